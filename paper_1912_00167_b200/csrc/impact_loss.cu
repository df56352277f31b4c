// Fused IMPACT loss + gradient kernels and their host entry points.
//
// One launch per call does every step of the learner's "compute policy and value network
// gradients" (Algorithm 1): log-probabilities under learner and target, truncated
// importance weights, the backward V-trace GAE-lambda recursion (Section 3.1), the
// target-worker-clipped, eps-clipped surrogate (Section 3.1, Appendix E), value / entropy /
// KL terms, the gradients, and the batch means.  Each input byte is read from HBM once and
// each output byte written once; nothing on this path is a matrix product, so no tensor
// cores are involved -- the kernel is bound by HBM bandwidth.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>

#include "impact.h"
#include "impact_device.cuh"
#include "impact_internal.h"

namespace impact {
namespace {

using dev::LossScalars;

struct TileGeometry {
    int tile_major;  // long trajectories in a persistent kernel: order of the grid's tiles (see place_of)
    long long B, T;
    long long nchunks;  // units of block-level work
    int G;              // whole trajectories per chunk (T <= NT), else 1
    int ntiles;         // tiles per trajectory (T > NT), else 1
};

struct CatParams {
    const void* learner_logits;
    const void* target_logits;
    const float* worker_logp;
    const int32_t* actions;
    const float* rewards;
    const float* discounts;
    const float* values;
    const float* bootstrap;
    float* loss_terms;
    void* dlogits;
    float* dvalues;
    float* vtarget;
    float* advantage;
    float* partials;
    unsigned int* counter;
    unsigned long long* tagged_rows;  // persistent kernel: rows of (value, launch tag) pairs, see dev::publish_tagged
    unsigned long long* tile_aggregates;  // persistent kernel, T > 128: two (value, launch tag) pairs per tile
    void* target_copy;  // persistent kernel: where the target logits are written as well (NULL = nowhere)
    const impact_loss_inputs* indirect;  // persistent kernel: device record that overrides the nine pointers above (NULL = none)
    TileGeometry geo;
    LossScalars k;
    int A, As;
};

struct GaussParams {
    const float* learner_mean;
    const float* learner_logstd;
    const float* target_mean;
    const float* target_logstd;
    const float* actions;
    const float* worker_logp;
    const float* rewards;
    const float* discounts;
    const float* values;
    const float* bootstrap;
    float* loss_terms;
    float* dmean;
    float* dlogstd;
    float* dvalues;
    float* vtarget;
    float* advantage;
    float* partials;
    unsigned int* counter;
    unsigned long long* tagged_rows;
    unsigned long long* tile_aggregates;
    TileGeometry geo;
    LossScalars k;
    int D, Ds;
};

// Where a tile sits: its first global row, how many rows, and each thread's (b, t).
struct TileRows {
    long long row0;
    int nrows;
};

template <int NT>
__device__ __forceinline__ TileRows tile_rows(const TileGeometry& g, long long chunk, int tile) {
    TileRows r;
    if (g.ntiles > 1) {
        const long long t0 = (long long)tile * NT;
        const long long left = g.T - t0;
        r.nrows = (int)(left < NT ? left : NT);
        r.row0 = chunk * g.T + t0;
    } else {
        const long long traj0 = chunk * g.G;
        long long ntraj = g.B - traj0;
        if (ntraj > g.G) ntraj = g.G;
        r.nrows = (int)(ntraj * g.T);
        r.row0 = traj0 * g.T;
    }
    return r;
}

// ------------------------------------------------------------------------------------------
// Categorical policy
// ------------------------------------------------------------------------------------------
// Element access for slabs that keep their storage type in shared memory.
template <typename ST> struct Elem;
template <> struct Elem<float> {
    static constexpr int kPerWord = 1;
    static __device__ __forceinline__ float ld(const unsigned char* slab, int i) { return reinterpret_cast<const float*>(slab)[i]; }
    static __device__ __forceinline__ void st(unsigned char* slab, int i, float x) { reinterpret_cast<float*>(slab)[i] = x; }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kPerWord = 2;
    static __device__ __forceinline__ float ld(const unsigned char* slab, int i) {
        return __uint_as_float((uint32_t)reinterpret_cast<const unsigned short*>(slab)[i] << 16);
    }
    static __device__ __forceinline__ void st(unsigned char* slab, int i, float x) {
        reinterpret_cast<__nv_bfloat16*>(slab)[i] = __float2bfloat16_rn(x);
    }
};

// Any action count (runtime A): the same tile protocol as the compile-time kernel below --
// bulk copies in, one thread per step, bulk copy out -- but rows stay in shared memory and
// are walked element by element in three passes.  The slabs keep their dense layout, so for
// row pitches that are a multiple of the bank width every thread would hit the same bank;
// instead thread r starts its walk at column (r * step) mod A and wraps, which spreads a
// warp's accesses over all banks without padding (order is irrelevant to max and sum).
template <typename LT, typename GT, int NT>
__global__ void __launch_bounds__(NT) impact_loss_categorical_kernel(const CatParams p) {
    grid_dependency_wait();
    constexpr float kLog2e = 1.4426950408889634f;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int A = p.A;
    const int in_row = A * (int)sizeof(LT), out_row = A * (int)sizeof(GT);
    unsigned char* const s0 = smem_raw;                // learner logits
    unsigned char* const s1 = smem_raw + NT * in_row;  // target logits
    unsigned char* const so = (sizeof(LT) == sizeof(GT)) ? s0 : smem_raw + 2 * NT * in_row;  // gradients
    __shared__ __align__(8) uint64_t bar;
    __shared__ float2 warp_agg[NT / 32];
    __shared__ float red[NT / 32][8];
    __shared__ float carry_s;
    __shared__ int is_last_s;

    const int tid = threadIdx.x;
    const LossScalars k = p.k;
    const TileGeometry g = p.geo;
    const LT* const zl = static_cast<const LT*>(p.learner_logits);
    const LT* const zt = static_cast<const LT*>(p.target_logits);
    GT* const dz = static_cast<GT*>(p.dlogits);
    const bool want_kl = (k.kl_coef != 0.0f);
    // first column of this thread's walk (see above): one storage word per row of skew when the
    // row pitch in words is even
    const int words = (A * (int)sizeof(LT)) / 4;
    const int rot = ((A * (int)sizeof(LT)) % 4 == 0 && words % 2 == 0) ? (tid * Elem<LT>::kPerWord) % A : 0;

    if (tid == 0) {
        dev::mbarrier_init(&bar, 1);
        is_last_s = 0;
    }
    __syncthreads();
    uint32_t parity = 0;

    float acc[dev::kNumSums], tsum[dev::kNumSums];
#pragma unroll
    for (int j = 0; j < dev::kNumSums; ++j) acc[j] = tsum[j] = 0.0f;

    for (long long chunk = blockIdx.x; chunk < g.nchunks; chunk += gridDim.x) {
        float carry = 0.0f;
        for (int tile = g.ntiles - 1; tile >= 0; --tile) {
            const bool final_tile = (tile == 0) && (chunk + gridDim.x >= g.nchunks);
            const TileRows tr = tile_rows<NT>(g, chunk, tile);
            const long long base = tr.row0 * A;
            const LT* const gl = zl + base;
            const LT* const gt = zt + base;
            GT* const gd = dz + base;
            const uint32_t in_bytes = (uint32_t)(tr.nrows * in_row), out_bytes = (uint32_t)(tr.nrows * out_row);
            const bool bulk_in = (((reinterpret_cast<uintptr_t>(gl) | reinterpret_cast<uintptr_t>(gt) | in_bytes) & 15u) == 0);
            const bool bulk_out = (((reinterpret_cast<uintptr_t>(gd) | out_bytes) & 15u) == 0);
            if (bulk_in) {
                if (tid == 0) {
                    dev::mbarrier_expect_tx(&bar, 2 * in_bytes);
                    dev::bulk_load(s0, gl, in_bytes, &bar);
                    dev::bulk_load(s1, gt, in_bytes, &bar);
                }
            } else {  // ragged or unaligned slab: plain element copies
                const int nelem = tr.nrows * A;
                for (int e = tid; e < nelem; e += NT) {
                    reinterpret_cast<LT*>(s0)[e] = gl[e];
                    reinterpret_cast<LT*>(s1)[e] = gt[e];
                }
            }

            const bool active = tid < tr.nrows;
            const long long row = tr.row0 + tid;
            dev::StepIn s;
            int a = 0;
            if (active) {
                long long b, t;
                if (g.ntiles > 1) { b = chunk; t = (long long)tile * NT + tid; }
                else if (g.G == 1) { b = chunk; t = tid; }
                else { const int q = tid / (int)g.T; b = chunk * g.G + q; t = tid - q * (int)g.T; }
                a = p.actions[row];
                a = a < 0 ? 0 : (a >= A ? A - 1 : a);
                s.l_worker = p.worker_logp[row];
                s.reward = p.rewards[row];
                s.discount = p.discounts[row];
                s.value = p.values[row];
                s.last_step = (t == g.T - 1);
                s.value_next = s.last_step ? p.bootstrap[b] : p.values[row + 1];
            }
            if (bulk_in) {
                if (tid < 32) {
                    if (!dev::mbarrier_wait(&bar, parity)) atomicExch(p.counter + 1, 1u);
                }
                parity ^= 1u;
            }
            __syncthreads();

            const int r0 = tid * A;  // first element of this thread's row
            float fa = 1.0f, fb = 0.0f;
            float m2_l = 0.0f, ln_s = 0.0f, inv_s = 0.0f, lse_t = 0.0f, ent = 0.0f, kl = 0.0f;
            bool truncated = false;
            if (active) {
                // target row: log-sum-exp
                float m = Elem<LT>::ld(s1, r0 + rot);
                for (int j = 1, c = rot; j < A; ++j) {
                    if (++c == A) c = 0;
                    m = fmaxf(m, Elem<LT>::ld(s1, r0 + c));
                }
                float sum = 0.0f;
                const float nm2 = -m * kLog2e;
                for (int j = 0, c = rot; j < A; ++j) {
                    sum += dev::exp2_fast(fmaf(Elem<LT>::ld(s1, r0 + c), kLog2e, nm2));
                    if (++c == A) c = 0;
                }
                lse_t = m + __logf(sum);
                s.l_target = Elem<LT>::ld(s1, r0 + a) - lse_t;
                // learner row: log-sum-exp and entropy, H = (m + ln S) - sum_j e_j z_j / S
                m = Elem<LT>::ld(s0, r0 + rot);
                for (int j = 1, c = rot; j < A; ++j) {
                    if (++c == A) c = 0;
                    m = fmaxf(m, Elem<LT>::ld(s0, r0 + c));
                }
                m2_l = m * kLog2e;
                sum = 0.0f;
                float sez = 0.0f;
                for (int j = 0, c = rot; j < A; ++j) {
                    const float z = Elem<LT>::ld(s0, r0 + c);
                    const float e = dev::exp2_fast(fmaf(z, kLog2e, -m2_l));
                    sum += e;
                    sez = fmaf(e, z, sez);
                    if (++c == A) c = 0;
                }
                ln_s = __logf(sum);
                inv_s = __frcp_rn(sum);
                ent = (m + ln_s) - sez * inv_s;
                s.l_theta = (Elem<LT>::ld(s0, r0 + a) - m) - ln_s;
                if (want_kl) {
                    const float lse_l = m + ln_s;
                    for (int j = 0, c = rot; j < A; ++j) {
                        const float lpt = Elem<LT>::ld(s1, r0 + c) - lse_t;
                        kl = fmaf(dev::exp2_fast(lpt * kLog2e), lpt - (Elem<LT>::ld(s0, r0 + c) - lse_l), kl);
                        if (++c == A) c = 0;
                    }
                }
                truncated = dev::recursion_map(s, k, fa, fb);
            }
            const float adv = dev::suffix_affine_scan<NT>(fa, fb, carry, warp_agg, s.adv_next);
            if (tid == 0) carry_s = adv;

            float surr = 0.0f, ratio = 0.0f, wpg = 0.0f;
            bool clipped = false;
            if (active) {
                wpg = dev::surrogate(s, k, adv, surr, ratio, clipped);
                tsum[0] += surr;
                tsum[1] = fmaf(0.5f * adv, adv, tsum[1]);
                tsum[2] += ent;
                tsum[3] += kl;
                tsum[4] += clipped ? 1.0f : 0.0f;
                tsum[5] += truncated ? 1.0f : 0.0f;
                tsum[6] += ratio;
            }
            unsigned int ticket = 0;
            if (final_tile) {
                dev::block_sums_stage1<NT>(tsum, red);
                __syncthreads();
                if (tid == 0) {
                    dev::block_sums_stage2<NT>(acc, red);
                    ticket = dev::publish_block_sums(acc, p.partials, p.counter);
                }
            }
            if (active) {
                // d total / d logit_j = [ wpg (pi_j - 1[j=a]) + ent_coef pi_j (lp_j + H)
                //                         + kl_coef (pi_j - pi_target_j) ] / M
                const float w1 = wpg * k.inv_M, ce = k.ent_coef * k.inv_M, ck = k.kl_coef * k.inv_M;
                const float h_off = ent - (m2_l * 0.6931471805599453f + ln_s);
                const float nlt2 = -lse_t * kLog2e;
                for (int j = 0, c = rot; j < A; ++j) {
                    const float z = Elem<LT>::ld(s0, r0 + c);
                    const float pi = dev::exp2_fast(fmaf(z, kLog2e, -m2_l)) * inv_s;
                    float gj = pi * fmaf(ce, z + h_off, w1);
                    if (want_kl) gj = fmaf(ck, pi - dev::exp2_fast(fmaf(Elem<LT>::ld(s1, r0 + c), kLog2e, nlt2)), gj);
                    if (c == a) gj -= w1;
                    Elem<GT>::st(so, r0 + c, gj);
                    if (++c == A) c = 0;
                }
                p.dvalues[row] = -k.vf_coef * k.inv_M * adv;  // V - Vhat = -A
                if (p.vtarget) p.vtarget[row] = s.value + adv;
                if (p.advantage) p.advantage[row] = adv;
            }
            if (bulk_out) dev::fence_async_shared();
            if (tid == 0 && final_tile) is_last_s = (ticket == gridDim.x - 1) ? 1 : 0;
            __syncthreads();
            carry = carry_s;
            if (bulk_out) {
                if (tid == 0) {
                    dev::bulk_store(gd, so, out_bytes);
                    if (!final_tile) dev::bulk_store_wait_read();
                }
            } else {
                const int nelem = tr.nrows * A;
                for (int i = tid; i < nelem; i += NT) gd[i] = reinterpret_cast<const GT*>(so)[i];
            }
            if (!final_tile) __syncthreads();
        }
    }
    if (is_last_s) dev::reduce_published_sums<NT>(p.partials, p.counter, p.loss_terms, k.vf_coef, k.ent_coef, k.kl_coef,
                                                   k.steps_total);
    if (tid == 0) dev::bulk_store_wait_read();
}

// ------------------------------------------------------------------------------------------
// Categorical policy, action count known at compile time: resident blocks that sweep a trajectory
// (long trajectories, many of them; every other batch goes to the persistent kernel further down)
// ------------------------------------------------------------------------------------------
// Same decomposition as the kernel above (128 steps per block, one thread per step), but:
//   * the two logits slabs of a tile arrive by ONE bulk asynchronous copy each, issued by a
//     single thread and signalled through an mbarrier, and the gradient slab leaves by one
//     bulk store: staging costs no per-element instructions and all of a tile's bytes are
//     in flight at once;
//   * the slabs keep their dense global layout in shared memory; a thread reads its row
//     with the widest vector access the row pitch allows, which is bank-conflict free for
//     the action counts compiled here (pitch/width odd);
//   * A is a template parameter and every loop is unrolled; rows are streamed pair by pair from
//     shared memory in each pass, so that few registers are live;
//   * the softmax runs on exp2 of pre-scaled differences (one multiply + one MUFU each).
// Five blocks per SM (<= 102 registers, no spills), two slab stages per block.
template <typename ST, int W> struct RowIO;

// Rows are handled as NP = ceil(W/2) pairs; for odd W the second lane of the last pair is
// padding (loaded as 0, never stored).
template <int W> struct RowIO<float, W> {
    static constexpr int NP = (W + 1) / 2;
    static __device__ __forceinline__ void load(const unsigned char* slab, int row, float2 (&v)[NP]) {
        const float* r = reinterpret_cast<const float*>(slab) + row * W;
        if constexpr (W % 4 == 0) {
#pragma unroll
            for (int j = 0; j < W / 4; ++j) {
                const float4 q = reinterpret_cast<const float4*>(r)[j];
                v[2 * j] = make_float2(q.x, q.y);
                v[2 * j + 1] = make_float2(q.z, q.w);
            }
        } else if constexpr (W % 2 == 0) {
#pragma unroll
            for (int j = 0; j < W / 2; ++j) v[j] = reinterpret_cast<const float2*>(r)[j];
        } else {
#pragma unroll
            for (int j = 0; j < W / 2; ++j) v[j] = make_float2(r[2 * j], r[2 * j + 1]);
            v[NP - 1] = make_float2(r[W - 1], 0.0f);
        }
    }
    static __device__ __forceinline__ void store(unsigned char* slab, int row, const float2 (&v)[NP]) {
        float* r = reinterpret_cast<float*>(slab) + row * W;
        if constexpr (W % 4 == 0) {
#pragma unroll
            for (int j = 0; j < W / 4; ++j)
                reinterpret_cast<float4*>(r)[j] = make_float4(v[2 * j].x, v[2 * j].y, v[2 * j + 1].x, v[2 * j + 1].y);
        } else if constexpr (W % 2 == 0) {
#pragma unroll
            for (int j = 0; j < W / 2; ++j) reinterpret_cast<float2*>(r)[j] = v[j];
        } else {
#pragma unroll
            for (int j = 0; j < W / 2; ++j) { r[2 * j] = v[j].x; r[2 * j + 1] = v[j].y; }
            r[W - 1] = v[NP - 1].x;
        }
    }
    // pair j of a row (elements 2j, 2j+1; the second lane of an odd row's last pair is 0)
    static __device__ __forceinline__ float2 load_pair(const unsigned char* slab, int row, int j) {
        const float* r = reinterpret_cast<const float*>(slab) + row * W;
        if constexpr (W % 2 == 0) return reinterpret_cast<const float2*>(r)[j];
        else return (2 * j + 1 < W) ? make_float2(r[2 * j], r[2 * j + 1]) : make_float2(r[2 * j], 0.0f);
    }
    static __device__ __forceinline__ void store_pair(unsigned char* slab, int row, int j, float2 v) {
        float* r = reinterpret_cast<float*>(slab) + row * W;
        if constexpr (W % 2 == 0) reinterpret_cast<float2*>(r)[j] = v;
        else { r[2 * j] = v.x; if (2 * j + 1 < W) r[2 * j + 1] = v.y; }
    }
    static __device__ __forceinline__ float at(const unsigned char* slab, int row, int col) {
        return reinterpret_cast<const float*>(slab)[row * W + col];
    }
    // Overwrites one element after `store` wrote the row; an explicit shared-memory store
    // keeps it ordered behind the vector stores to the same bytes.
    static __device__ __forceinline__ void put(unsigned char* slab, int row, int col, float x) {
        asm volatile("st.shared.f32 [%0], %1;" ::"r"(dev::smem_addr(slab) + (uint32_t)(row * W + col) * 4u), "f"(x)
                     : "memory");
    }
};

template <int W> struct RowIO<__nv_bfloat16, W> {
    static constexpr int NP = (W + 1) / 2;
    static __device__ __forceinline__ float widen(unsigned short h) { return __uint_as_float((uint32_t)h << 16); }
    static __device__ __forceinline__ void load(const unsigned char* slab, int row, float2 (&v)[NP]) {
        if constexpr (W % 2 == 0) {
            const uint32_t* r = reinterpret_cast<const uint32_t*>(slab) + row * (W / 2);
#pragma unroll
            for (int j = 0; j < W / 2; ++j) {
                const uint32_t w = r[j];
                v[j] = make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
            }
        } else {
            const unsigned short* r = reinterpret_cast<const unsigned short*>(slab) + row * W;
#pragma unroll
            for (int j = 0; j < W / 2; ++j) v[j] = make_float2(widen(r[2 * j]), widen(r[2 * j + 1]));
            v[NP - 1] = make_float2(widen(r[W - 1]), 0.0f);
        }
    }
    static __device__ __forceinline__ void store(unsigned char* slab, int row, const float2 (&v)[NP]) {
        if constexpr (W % 2 == 0) {
            uint32_t* r = reinterpret_cast<uint32_t*>(slab) + row * (W / 2);
#pragma unroll
            for (int j = 0; j < W / 2; ++j) r[j] = dev::Pack<__nv_bfloat16>::two(v[j].x, v[j].y);
        } else {
            __nv_bfloat16* r = reinterpret_cast<__nv_bfloat16*>(slab) + row * W;
#pragma unroll
            for (int j = 0; j < W / 2; ++j) {
                r[2 * j] = __float2bfloat16_rn(v[j].x);
                r[2 * j + 1] = __float2bfloat16_rn(v[j].y);
            }
            r[W - 1] = __float2bfloat16_rn(v[NP - 1].x);
        }
    }
    static __device__ __forceinline__ float2 load_pair(const unsigned char* slab, int row, int j) {
        if constexpr (W % 2 == 0) {
            const uint32_t w = reinterpret_cast<const uint32_t*>(slab)[row * (W / 2) + j];
            return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
        } else {
            const unsigned short* r = reinterpret_cast<const unsigned short*>(slab) + row * W;
            return (2 * j + 1 < W) ? make_float2(widen(r[2 * j]), widen(r[2 * j + 1])) : make_float2(widen(r[2 * j]), 0.0f);
        }
    }
    static __device__ __forceinline__ void store_pair(unsigned char* slab, int row, int j, float2 v) {
        if constexpr (W % 2 == 0) {
            reinterpret_cast<uint32_t*>(slab)[row * (W / 2) + j] = dev::Pack<__nv_bfloat16>::two(v.x, v.y);
        } else {
            __nv_bfloat16* r = reinterpret_cast<__nv_bfloat16*>(slab) + row * W;
            r[2 * j] = __float2bfloat16_rn(v.x);
            if (2 * j + 1 < W) r[2 * j + 1] = __float2bfloat16_rn(v.y);
        }
    }
    static __device__ __forceinline__ float at(const unsigned char* slab, int row, int col) {
        return widen(reinterpret_cast<const unsigned short*>(slab)[row * W + col]);
    }
    static __device__ __forceinline__ void put(unsigned char* slab, int row, int col, float x) {
        const unsigned short h = __bfloat16_as_ushort(__float2bfloat16_rn(x));
        asm volatile("st.shared.u16 [%0], %1;" ::"r"(dev::smem_addr(slab) + (uint32_t)(row * W + col) * 2u), "h"(h)
                     : "memory");
    }
};

constexpr int kRegTileRows = 128;

// Shared memory of the register-resident kernel, per pipeline stage: the two input slabs,
// plus a separate gradient slab only when gradients and logits differ in element size
// (otherwise each thread's gradient row replaces its own logits row).
template <typename LT, typename GT, int A>
__host__ __device__ constexpr size_t reg_kernel_stage_bytes() {
    constexpr size_t in_row = A * sizeof(LT), out_row = A * sizeof(GT);
    return kRegTileRows * (2 * in_row + (sizeof(LT) == sizeof(GT) ? 0 : out_row));
}
template <typename LT, typename GT, int A>
constexpr size_t reg_kernel_smem() {
    return 2 * reg_kernel_stage_bytes<LT, GT, A>();  // two stages
}

template <typename LT, typename GT, int A>
__global__ void __launch_bounds__(kRegTileRows, 5) impact_loss_categorical_reg_kernel(const CatParams p) {
    grid_dependency_wait();
    constexpr int NT = kRegTileRows;
    constexpr int NP = (A + 1) / 2;  // pairs per row: Blackwell's packed fp32 add / mul / fma work on two lanes at once
    constexpr bool kOdd = (A & 1) != 0;
    constexpr int kInRow = A * (int)sizeof(LT), kOutRow = A * (int)sizeof(GT);
    constexpr int kStageBytes = (int)reg_kernel_stage_bytes<LT, GT, A>();
    constexpr float kLog2e = 1.4426950408889634f;
    // Two stages of slabs: while a tile is being worked on, the block's next tile is already
    // streaming into the other stage (slabs by bulk copy, per-step scalars into registers).
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t bar[2];
    __shared__ float2 warp_agg[NT / 32];
    __shared__ float red[NT / 32][8];
    __shared__ float carry_s;
    __shared__ int is_last_s;

    const int tid = threadIdx.x;
    const LossScalars k = p.k;
    const TileGeometry g = p.geo;
    const LT* const zl = static_cast<const LT*>(p.learner_logits);
    const LT* const zt = static_cast<const LT*>(p.target_logits);
    GT* const dz = static_cast<GT*>(p.dlogits);
    const bool want_kl = (k.kl_coef != 0.0f);
    const float2 log2e2 = make_float2(kLog2e, kLog2e);

    if (tid == 0) {
        dev::mbarrier_init(&bar[0], 1);
        dev::mbarrier_init(&bar[1], 1);
        is_last_s = 0;
    }
    __syncthreads();

    // This block's work: chunks blockIdx.x, blockIdx.x + gridDim.x, ...; within a chunk the tiles
    // of a long trajectory from the last one backwards.  Iteration `it` of the block is
    // (chunk, tile) = (blockIdx.x + (it / ntiles) * gridDim.x, ntiles - 1 - it % ntiles).
    const long long n_iter = ((g.nchunks - blockIdx.x + gridDim.x - 1) / gridDim.x) * g.ntiles;

    struct Tile {
        long long chunk, row0;
        int tile, nrows;
        bool bulk_in;
    };
    auto tile_of = [&](long long it) {
        Tile t;
        // (no 64-bit division on the common path: one tile per trajectory)
        const long long ci = (g.ntiles == 1) ? it : (long long)((unsigned long long)it / (unsigned int)g.ntiles);
        t.chunk = blockIdx.x + ci * gridDim.x;
        t.tile = g.ntiles - 1 - (int)(it - ci * g.ntiles);
        const TileRows tr = tile_rows<NT>(g, t.chunk, t.tile);
        t.row0 = tr.row0;
        t.nrows = tr.nrows;
        const uintptr_t a0 = reinterpret_cast<uintptr_t>(zl + tr.row0 * A), a1 = reinterpret_cast<uintptr_t>(zt + tr.row0 * A);
        t.bulk_in = (((a0 | a1 | (uintptr_t)(tr.nrows * kInRow)) & 15u) == 0);
        return t;
    };
    // Start the slab copies of a tile into a stage (whose previous contents are no longer needed).
    auto fill_stage = [&](const Tile& t, int stage) {
        unsigned char* const d0 = smem_raw + stage * kStageBytes;
        unsigned char* const d1 = d0 + NT * kInRow;
        const LT* const gl = zl + t.row0 * A;
        const LT* const gt = zt + t.row0 * A;
        if (t.bulk_in) {
            if (tid == 0) {
                const uint32_t bytes = (uint32_t)t.nrows * kInRow;
                dev::mbarrier_expect_tx(&bar[stage], 2 * bytes);
                dev::bulk_load(d0, gl, bytes, &bar[stage]);
                dev::bulk_load(d1, gt, bytes, &bar[stage]);
            }
        } else {  // ragged or unaligned slab: plain element copies
            const int nelem = t.nrows * A;
            for (int e = tid; e < nelem; e += NT) {
                reinterpret_cast<LT*>(d0)[e] = gl[e];
                reinterpret_cast<LT*>(d1)[e] = gt[e];
            }
        }
    };
    // Per-step scalars of a tile, straight from global memory (coalesced).
    struct StepRaw {
        int a;
        float l_worker, reward, discount, value, value_next;
        bool last_step;
    };
    auto load_scalars = [&](const Tile& t) {
        StepRaw r;
        r.a = 0; r.l_worker = 0.f; r.reward = 0.f; r.discount = 0.f; r.value = 0.f; r.value_next = 0.f;
        r.last_step = false;
        if (tid < t.nrows) {
            const long long row = t.row0 + tid;
            long long b, ts;
            if (g.ntiles > 1) { b = t.chunk; ts = (long long)t.tile * NT + tid; }
            else if (g.G == 1) { b = t.chunk; ts = tid; }
            else { const int q = tid / (int)g.T; b = t.chunk * g.G + q; ts = tid - q * (int)g.T; }
            int a = p.actions[row];
            r.a = a < 0 ? 0 : (a >= A ? A - 1 : a);
            r.l_worker = p.worker_logp[row];
            r.reward = p.rewards[row];
            r.discount = p.discounts[row];
            r.value = p.values[row];
            r.last_step = (ts == g.T - 1);
            r.value_next = r.last_step ? p.bootstrap[b] : p.values[row + 1];
        }
        return r;
    };

    float acc[dev::kNumSums], tsum[dev::kNumSums];
#pragma unroll
    for (int j = 0; j < dev::kNumSums; ++j) acc[j] = tsum[j] = 0.0f;

    Tile cur_tile = tile_of(0);
    fill_stage(cur_tile, 0);
    StepRaw cur = load_scalars(cur_tile);
    uint32_t parity_bits = 0;  // bit s: phase parity the next wait on bar[s] expects
    float carry = 0.0f;

    for (long long it = 0; it < n_iter; ++it) {
        {
            const int stage = (int)(it & 1);
            const bool final_tile = (it + 1 == n_iter);
            const Tile tl = cur_tile;
            if (tl.tile == g.ntiles - 1) carry = 0.0f;  // a new trajectory starts (from its end)
            // prefetch: the other stage was released by the barrier that ended the previous tile
            Tile next_tile = tl;
            StepRaw nxt = cur;
            if (!final_tile) {
                next_tile = tile_of(it + 1);
                fill_stage(next_tile, stage ^ 1);
                nxt = load_scalars(next_tile);
            }

            unsigned char* const s0 = smem_raw + stage * kStageBytes;  // learner logits
            unsigned char* const s1 = s0 + NT * kInRow;                // target logits
            // gradient rows: over the thread's own logits row when the element sizes agree
            unsigned char* const so = (sizeof(LT) == sizeof(GT)) ? s0 : s0 + 2 * NT * kInRow;
            GT* const gd = dz + tl.row0 * A;
            const uint32_t out_bytes = (uint32_t)tl.nrows * kOutRow;
            const bool bulk_out = (((reinterpret_cast<uintptr_t>(gd) | out_bytes) & 15u) == 0);
            const bool active = tid < tl.nrows;
            const long long row = tl.row0 + tid;
            const int a = cur.a;
            dev::StepIn s;
            s.l_worker = cur.l_worker;
            s.reward = cur.reward;
            s.discount = cur.discount;
            s.value = cur.value;
            s.value_next = cur.value_next;
            s.last_step = cur.last_step;

            if (tl.bulk_in) {
                // one warp watches the mbarrier; the others sleep at the block barrier
                if (tid < 32) {
                    if (!dev::mbarrier_wait(&bar[stage], (parity_bits >> stage) & 1u)) atomicExch(p.counter + 1, 1u);
                }
                parity_bits ^= (1u << stage);
            }
            __syncthreads();

            float fa = 1.0f, fb = 0.0f;
            // Rows are streamed pair by pair from shared memory in every pass and nothing row-sized is
            // held in registers (not within a pass, not across the scan): shared-memory reads are cheap
            // here, registers are what limits how many rows an SM works on at once.
            float m2_l = 0.0f, ln_s = 0.0f, inv_s = 0.0f, lse_t = 0.0f, ent = 0.0f, kl = 0.0f;
            bool truncated = false;
            if (active) {
                {   // target row: only its log-sum-exp and the taken action's logit are needed
                    float2 mx = RowIO<LT, A>::load_pair(s1, tid, 0);
                    if (kOdd && NP == 1) mx.y = mx.x;
#pragma unroll
                    for (int j = 1; j < NP; ++j) {
                        float2 v = RowIO<LT, A>::load_pair(s1, tid, j);
                        if (kOdd && j == NP - 1) v.y = v.x;
                        mx.x = fmaxf(mx.x, v.x);
                        mx.y = fmaxf(mx.y, v.y);
                    }
                    const float m = fmaxf(mx.x, mx.y);
                    const float2 neg_m2 = make_float2(-m * kLog2e, -m * kLog2e);
                    float2 sum2 = make_float2(0.0f, 0.0f);
#pragma unroll
                    for (int j = 0; j < NP; ++j) {
                        const float2 t2 = __ffma2_rn(RowIO<LT, A>::load_pair(s1, tid, j), log2e2, neg_m2);  // (z - m) log2 e
                        float2 ex = make_float2(dev::exp2_fast(t2.x), dev::exp2_fast(t2.y));
                        if (kOdd && j == NP - 1) ex.y = 0.0f;
                        sum2 = __fadd2_rn(sum2, ex);
                    }
                    lse_t = m + __logf(sum2.x + sum2.y);
                    s.l_target = RowIO<LT, A>::at(s1, tid, a) - lse_t;
                }
                float2 mx = RowIO<LT, A>::load_pair(s0, tid, 0);
                if (kOdd && NP == 1) mx.y = mx.x;
#pragma unroll
                for (int j = 1; j < NP; ++j) {
                    float2 v = RowIO<LT, A>::load_pair(s0, tid, j);
                    if (kOdd && j == NP - 1) v.y = v.x;
                    mx.x = fmaxf(mx.x, v.x);
                    mx.y = fmaxf(mx.y, v.y);
                }
                const float m = fmaxf(mx.x, mx.y);
                m2_l = m * kLog2e;
                const float2 neg_m2 = make_float2(-m2_l, -m2_l);
                float2 sum2 = make_float2(0.0f, 0.0f), sez2 = make_float2(0.0f, 0.0f);
#pragma unroll
                for (int j = 0; j < NP; ++j) {
                    const float2 z = RowIO<LT, A>::load_pair(s0, tid, j);
                    const float2 t2 = __ffma2_rn(z, log2e2, neg_m2);
                    float2 ex = make_float2(dev::exp2_fast(t2.x), dev::exp2_fast(t2.y));
                    if (kOdd && j == NP - 1) ex.y = 0.0f;
                    sum2 = __fadd2_rn(sum2, ex);
                    sez2 = __ffma2_rn(ex, z, sez2);
                }
                const float sum = sum2.x + sum2.y;
                ln_s = __logf(sum);
                inv_s = __frcp_rn(sum);
                // H = -sum_j pi_j lp_j = (m + ln S) - sum_j e_j z_j / S
                ent = (m + ln_s) - (sez2.x + sez2.y) * inv_s;
                s.l_theta = (RowIO<LT, A>::at(s0, tid, a) - m) - ln_s;
                if (want_kl) {
                    const float lse_l = m + ln_s;
#pragma unroll
                    for (int j = 0; j < A; ++j) {
                        const float lpt = RowIO<LT, A>::at(s1, tid, j) - lse_t;
                        kl = fmaf(dev::exp2_fast(lpt * kLog2e), lpt - (RowIO<LT, A>::at(s0, tid, j) - lse_l), kl);
                    }
                }
                truncated = dev::recursion_map(s, k, fa, fb);
            }
            const float adv = dev::suffix_affine_scan<NT>(fa, fb, carry, warp_agg, s.adv_next);
            if (tid == 0) carry_s = adv;

            float surr = 0.0f, ratio = 0.0f, wpg = 0.0f;
            bool clipped = false;
            if (active) wpg = dev::surrogate(s, k, adv, surr, ratio, clipped);
            // each thread keeps its own running sums over the block's tiles; they are added across
            // the block once, in the last tile, and published right away so that the round trip
            // hides behind the epilogue
            if (active) {
                tsum[0] += surr;
                tsum[1] = fmaf(0.5f * adv, adv, tsum[1]);
                tsum[2] += ent;
                tsum[3] += kl;
                tsum[4] += clipped ? 1.0f : 0.0f;
                tsum[5] += truncated ? 1.0f : 0.0f;
                tsum[6] += ratio;
            }
            unsigned int ticket = 0;
            if (final_tile) {
                dev::block_sums_stage1<NT>(tsum, red);
                __syncthreads();
                if (tid == 0) {
                    dev::block_sums_stage2<NT>(acc, red);
                    ticket = dev::publish_block_sums(acc, p.partials, p.counter);
                }
            }

            if (active) {
                // d total / d logit_j = [ wpg (pi_j - 1[j=a]) + ent_coef pi_j (lp_j + H)
                //                         + kl_coef (pi_j - pi_target_j) ] / M
                // with pi_j = 2^(z_j log2 e - m log2 e) / S and lp_j + H = z_j + (H - m - ln S)
                const float w1 = wpg * k.inv_M, ce = k.ent_coef * k.inv_M, ck = k.kl_coef * k.inv_M;
                const float h_off = ent - (m2_l * 0.6931471805599453f + ln_s);
                const float2 inv_s2 = make_float2(inv_s, inv_s), hoff2 = make_float2(h_off, h_off);
                const float2 ce2 = make_float2(ce, ce), w12 = make_float2(w1, w1);
                const float2 neg_m2 = make_float2(-m2_l, -m2_l);
                const float2 ck2 = make_float2(ck, ck);
                const float2 neg_lse_t2 = make_float2(-lse_t * kLog2e, -lse_t * kLog2e);
#pragma unroll
                for (int j = 0; j < NP; ++j) {
                    const float2 z = RowIO<LT, A>::load_pair(s0, tid, j);
                    const float2 t2 = __ffma2_rn(z, log2e2, neg_m2);
                    const float2 pi2 = __fmul2_rn(make_float2(dev::exp2_fast(t2.x), dev::exp2_fast(t2.y)), inv_s2);
                    float2 g2 = __fmul2_rn(pi2, __ffma2_rn(ce2, __fadd2_rn(z, hoff2), w12));
                    if (want_kl) {
                        const float2 tt = __ffma2_rn(RowIO<LT, A>::load_pair(s1, tid, j), log2e2, neg_lse_t2);
                        const float2 npt = make_float2(-dev::exp2_fast(tt.x), -dev::exp2_fast(tt.y));
                        g2 = __ffma2_rn(ck2, __fadd2_rn(pi2, npt), g2);
                    }
                    RowIO<GT, A>::store_pair(so, tid, j, g2);
                }
                // the taken action's entry, from its own log-probability
                const float pi_a = dev::exp2_fast(s.l_theta * kLog2e);
                float g_a = fmaf(pi_a, fmaf(ce, s.l_theta + ent, w1), -w1);
                if (want_kl) g_a = fmaf(ck, pi_a - dev::exp2_fast(s.l_target * kLog2e), g_a);
                p.dvalues[row] = -k.vf_coef * k.inv_M * adv;  // V - Vhat = -A
                if (p.vtarget) p.vtarget[row] = s.value + adv;
                if (p.advantage) p.advantage[row] = adv;
                RowIO<GT, A>::put(so, tid, a, g_a);
            }
            if (bulk_out) dev::fence_async_shared();
            if (tid == 0 && final_tile) is_last_s = (ticket == gridDim.x - 1) ? 1 : 0;
            __syncthreads();
            carry = carry_s;
            if (bulk_out) {
                if (tid == 0) {
                    dev::bulk_store(gd, so, out_bytes);
                    if (!final_tile) dev::bulk_store_wait_read();  // the last store drains at the very end
                }
            } else {
                const int nelem = tl.nrows * A;
                for (int i = tid; i < nelem; i += NT) gd[i] = reinterpret_cast<const GT*>(so)[i];
            }
            if (!final_tile) __syncthreads();  // this stage, the sums and the carry are free again
            cur_tile = next_tile;
            cur = nxt;
        }
    }
    if (is_last_s) dev::reduce_published_sums<NT>(p.partials, p.counter, p.loss_terms, k.vf_coef, k.ent_coef, k.kl_coef,
                                                   k.steps_total);
    if (tid == 0) dev::bulk_store_wait_read();  // shared memory must outlive the store's reads
}

// ------------------------------------------------------------------------------------------
// Categorical policy, persistent warp-specialised form (trajectories of at most 128 steps)
// ------------------------------------------------------------------------------------------
// One block per SM.  A producer warp streams the block's tiles (blockIdx.x, + gridDim.x, ...)
// through a ring of shared-memory stages, keeping a fixed number of tiles in flight, so that
// tiles land one after the other from the first microseconds on instead of all at the end;
// C consumer groups of 128 threads (one thread per step, as above) each take every C-th tile
// as it lands, and every warp sends its own 32 gradient rows off by a bulk store while later
// tiles are still arriving.  Loading, arithmetic and storing overlap inside one launch: a
// B*T = 131072 batch (seven tiles per SM) takes 9.7 us against 12.5 us for resident blocks
// that each load, compute and store one tile, and batches of a million steps and more run at
// the speed of a device-to-device copy.
//
// Barriers: full[s] (one arrival + the bytes of the two slabs) says stage s holds a tile;
// empty[s] (one arrival per consumer warp, after that warp's store has finished reading the
// stage) says it may be refilled.  Every wait is bounded; a wait that gives up raises the
// workspace's error word and the block's abort flag, after which nobody waits any more and
// the block runs to its end on whatever the stages hold.
// Where the n-th tile of a block of a persistent kernel sits: first row, rows, first trajectory, and (long
// trajectories) the tile's number counted from its trajectory's end.
struct Place {
    long long row0, traj;
    int nrows, r;
};
template <bool kLong, int NT>
__device__ __forceinline__ Place tile_place(const TileGeometry& g, int n, int rows_full, long long total_rows) {
    Place pl;
    const long long gt_ = (long long)blockIdx.x + (long long)n * gridDim.x;
    if (kLong) {
        if (g.tile_major) {  // the last tiles of all trajectories first, then the tiles before them, ...
            pl.r = (int)((unsigned long long)gt_ / (unsigned long long)g.B);
            pl.traj = gt_ - (long long)pl.r * g.B;
        } else {  // trajectory by trajectory, each from its last tile backwards
            pl.traj = (long long)((unsigned long long)gt_ / (unsigned int)g.ntiles);
            pl.r = (int)(gt_ - pl.traj * g.ntiles);
        }
        const long long t0 = (long long)(g.ntiles - 1 - pl.r) * NT;
        const long long left = g.T - t0;
        pl.nrows = left < NT ? (int)left : NT;
        pl.row0 = pl.traj * g.T + t0;
    } else {
        pl.row0 = gt_ * rows_full;
        pl.traj = gt_ * g.G;
        const long long left = total_rows - pl.row0;
        pl.nrows = left < rows_full ? (int)left : rows_full;
        pl.r = 0;
    }
    return pl;
}

// A slab of the persistent kernels in shared memory: NT rows of `row_bytes`, plus 32 bytes of padding, because a
// tile's rows sit at the same offset inside their 16-byte granule as in global memory (0..15 bytes after the
// slab's start) and the copy that brings them is widened to whole granules (see dev::widen_range).
__host__ __device__ constexpr size_t ws_slab_pitch(size_t nt, size_t row_bytes) { return nt * row_bytes + 32; }

template <typename LT, typename GT, int A, int NT>
__host__ __device__ constexpr size_t ws_stage_bytes() {
    constexpr size_t in_row = A * sizeof(LT), out_row = A * sizeof(GT);
    constexpr size_t raw = 2 * ws_slab_pitch(NT, in_row) + (sizeof(LT) == sizeof(GT) ? 0 : ws_slab_pitch(NT, out_row));
    return (raw + 127) / 128 * 128;
}

// The same placement with the tile size and the form of the grid as run-time values (the companion kernel that
// only prefetches, below).
__device__ __forceinline__ Place tile_place_rt(const TileGeometry& g, int n, int rows_full, long long total_rows,
                                               bool is_long, int nt) {
    Place pl;
    const long long gt_ = (long long)blockIdx.x + (long long)n * gridDim.x;
    if (is_long) {
        if (g.tile_major) {
            pl.r = (int)((unsigned long long)gt_ / (unsigned long long)g.B);
            pl.traj = gt_ - (long long)pl.r * g.B;
        } else {
            pl.traj = (long long)((unsigned long long)gt_ / (unsigned int)g.ntiles);
            pl.r = (int)(gt_ - pl.traj * g.ntiles);
        }
        const long long t0 = (long long)(g.ntiles - 1 - pl.r) * nt;
        const long long left = g.T - t0;
        pl.nrows = left < nt ? (int)left : nt;
        pl.row0 = pl.traj * g.T + t0;
    } else {
        pl.row0 = gt_ * rows_full;
        pl.traj = gt_ * g.G;
        const long long left = total_rows - pl.row0;
        pl.nrows = left < rows_full ? (int)left : rows_full;
        pl.r = 0;
    }
    return pl;
}

// ---- early prefetch -------------------------------------------------------------------------------------------
// What a block of a persistent kernel will read, as a list of row-major arrays: the first tiles of every block
// are asked for in L2 before the launch's stream dependency has resolved.  A prefetch changes nothing that a
// program can observe (L2 is where the device's writes meet, so a later write to these addresses is not lost);
// it only moves the wait for HBM from the start of this launch into the end of the one before it.
constexpr int kMaxPrefetchArrays = 10;
struct PrefetchList {
    const void* base[kMaxPrefetchArrays];
    int row_bytes[kMaxPrefetchArrays];
    int n_arrays;
    int n_tiles_max;  // tiles of a block that are asked for (from its first)
    int nt;           // rows per tile
    int is_long;
    TileGeometry geo;
};

// Run by one warp: tile after tile in the order the block will want them, lane a asking for array a's rows of
// the tile, so that the memory system sees the requests in that order too.
__device__ __forceinline__ void prefetch_block_tiles(const PrefetchList& pf) {
    const int lane = threadIdx.x & 31;
    const TileGeometry& g = pf.geo;
    const long long total_tiles = pf.is_long ? g.nchunks * g.ntiles : g.nchunks;
    int n_tiles = (int)((total_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x);
    if (n_tiles > pf.n_tiles_max) n_tiles = pf.n_tiles_max;
    const int rows_full = pf.is_long ? pf.nt : g.G * (int)g.T;
    const long long total_rows = g.B * g.T;
    const void* base = nullptr;
    long long pitch = 0;
#pragma unroll
    for (int a = 0; a < kMaxPrefetchArrays; ++a)
        if (lane == a && a < pf.n_arrays) { base = pf.base[a]; pitch = pf.row_bytes[a]; }
    for (int n = 0; n < n_tiles; ++n) {
        const Place pc = tile_place_rt(g, n, rows_full, total_rows, pf.is_long != 0, pf.nt);
        if (base) dev::prefetch_range_l2(base, pc.row0 * pitch, (uint32_t)(pc.nrows * pitch), total_rows * pitch);
    }
}

// The companion of a loss launch: enqueued right before it, it becomes resident next to the blocks of whatever
// kernel is still running on the stream (it needs one warp and no shared memory per block), asks L2 for the
// loss launch's first tiles, and only then waits for the stream's previous kernel -- which keeps stream order
// exact for the loss kernel behind it, whose own dependency is this kernel.
__global__ void __launch_bounds__(32) impact_prefetch_kernel(const __grid_constant__ PrefetchList pf) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    prefetch_block_tiles(pf);
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
constexpr int ws_tile_rows(int A) { return A > 32 ? 64 : 128; }
constexpr int kWsMaxStages = 24;
constexpr int kWsGroups = 4;  // consumer groups per block at least (16 consumer warps + the producer warp)

// Row passes of one step, shared by the kernels with a compile-time action count.  `zr` / `tr`
// point at the thread's learner / target row in shared memory.
template <typename LT, int A>
struct RowMath {
    static constexpr int NP = (A + 1) / 2;
    static constexpr bool kOdd = (A & 1) != 0;
    static constexpr float kLog2e = 1.4426950408889634f;

    // log2-sum-exp (base 2, of z log2 e) of a row; optionally keeps the exponentials and sum_j e_j z_j
    template <bool kKeep>
    static __device__ __forceinline__ float lse2(const unsigned char* slab, int row, float2 (&e)[NP], float& m2, float& sum,
                                                 float& sez) {
        float2 v[NP];
        RowIO<LT, A>::load(slab, row, v);
        float m0, m1;
        {
            const float y0 = (kOdd && NP == 1) ? v[0].x : v[0].y;
            m0 = fmaxf(v[0].x, y0);
            m1 = m0;
        }
#pragma unroll
        for (int j = 1; j < NP; ++j) {
            const float y = (kOdd && j == NP - 1) ? v[j].x : v[j].y;
            if (j & 1) m1 = fmaxf(m1, fmaxf(v[j].x, y));
            else m0 = fmaxf(m0, fmaxf(v[j].x, y));
        }
        m2 = fmaxf(m0, m1) * kLog2e;
        const float2 neg_m2 = make_float2(-m2, -m2), log2e2 = make_float2(kLog2e, kLog2e);
        float2 sum2 = make_float2(0.0f, 0.0f), sez2 = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int j = 0; j < NP; ++j) {
            const float2 t2 = __ffma2_rn(v[j], log2e2, neg_m2);  // (z - m) log2 e
            float2 ex = make_float2(dev::exp2_fast(t2.x), dev::exp2_fast(t2.y));
            if (kOdd && j == NP - 1) ex.y = 0.0f;
            sum2 = __fadd2_rn(sum2, ex);
            if (kKeep) {
                e[j] = ex;
                sez2 = __ffma2_rn(ex, v[j], sez2);
            }
        }
        sum = sum2.x + sum2.y;
        sez = sez2.x + sez2.y;
        return m2 + dev::log2_fast(sum);
    }
};

// kPlain: the configuration of the paper's experiments -- no KL term, the clipped surrogate with the
// default ratio and importance weights, no optional outputs -- with those branches compiled out.
//
// kLong: trajectories longer than a tile.  The grid's tiles are numbered either trajectory by trajectory, each from
// its END backwards (few tiles in all: the tiles of one trajectory go to neighbouring blocks, are contiguous in
// memory and are worked on at the same time), or tile-major (many: all trajectories' last tiles first, then the tiles
// before them, ..., so that the aggregates a tile needs were published a round earlier and one early look finds
// them).  The recursion crosses tiles through their affine aggregates: a tile composes its 128 maps into one
// (a, b), publishes it as two (value, launch tag) pairs, reads the aggregates of the later tiles of its
// trajectory -- all of them at once, a lane each -- and composes them, applied to 0, into the value that enters
// its own last step.  Nothing waits on a chain of tiles: every tile waits only for aggregates, which need
// nothing but their own tile's rows, and only of tiles with a smaller number, which no block starts later
// than the waiting one.
//
// NT: steps per tile = threads per consumer group (128; 64 for A = 64, whose rows are four times as long).
// Rows wider than 32 actions are not held in registers: every pass streams the row from shared memory, the
// gradient pass forms the exponentials again, and thread r starts its walk at pair r mod (A/2), because a row
// pitch of 256 bytes would otherwise put all threads of a warp on the same banks.
struct LossInputPointers {
    const void* learner_logits;
    const void* target_logits;
    const float* worker_logp;
    const int32_t* actions;
    const float* rewards;
    const float* discounts;
    const float* values;
    const float* bootstrap;
    void* target_copy;
};
// The record of impact_buffer_device_step, read past L1 (an earlier launch may have left an older version there).
__device__ __forceinline__ LossInputPointers fetch_loss_inputs(const impact_loss_inputs* rec) {
    const ulonglong2* q = reinterpret_cast<const ulonglong2*>(rec);
    const ulonglong2 a = __ldcg(q), b = __ldcg(q + 1), c = __ldcg(q + 2), d = __ldcg(q + 3);
    const unsigned long long e = __ldcg(reinterpret_cast<const unsigned long long*>(q + 4));
    LossInputPointers in;
    in.learner_logits = reinterpret_cast<const void*>(a.x);
    in.target_logits = reinterpret_cast<const void*>(a.y);
    in.worker_logp = reinterpret_cast<const float*>(b.x);
    in.actions = reinterpret_cast<const int32_t*>(b.y);
    in.rewards = reinterpret_cast<const float*>(c.x);
    in.discounts = reinterpret_cast<const float*>(c.y);
    in.values = reinterpret_cast<const float*>(d.x);
    in.bootstrap = reinterpret_cast<const float*>(d.y);
    in.target_copy = reinterpret_cast<void*>(e);
    return in;
}

// Barrier protocol of the persistent kernels (S stages, at most W tiles in flight, lanes <= S - W):
//   full[s]     one arrival (a producer lane's, with the bytes the tile's two copies will deliver): stage s holds
//               the rows of its current tile.
//   empty[s]    one arrival per consumer warp, after that warp's stores have finished reading the stage.
// A wait names a phase by its PARITY, which is only unambiguous while the waiter is at most one phase ahead of the
// barrier: asked about phase k while phase k-1 is still open, the barrier answers "complete".  The producer
// therefore issues tiles STRICTLY in order, and tile n only after (a) tile n-W has landed and
// (b) every consumer warp has released tile n-S.  From that:
//   * consumer of tile n waits on full[n % S] for phase n/S.  It got there after consuming tile n-C, so n-C was
//     issued, so (in order) tile n-S+W <= n-C was issued, so by (a) tile n-S -- phase n/S - 1 of the same stage --
//     had landed: the barrier is in phase n/S or later.  It cannot be beyond n/S + 1 open, because tile n+S is not
//     issued before this consumer releases tile n (b).  (This is where S >= W + C is needed.)
//   * producer's look at full[(n-W) % S] for phase (n-W)/S: tile n-W was issued, so by (b) tile n-W-S was consumed,
//     hence had landed: phase (n-W)/S - 1 is complete; tile n-W+S > n is not issued yet.
//   * producer's look at empty[n % S] for phase n/S - 1: tile n-S was issued, so by (b) phase n/S - 2 is complete;
//     phase n/S needs the consumers of tile n, which is not issued yet.
// Without the in-order rule (lanes that found their own tile ready first went first) the first argument fails for
// tiles of one round: a consumer could be handed a stage whose previous tile had not landed, read stale rows,
// release the stage early, and the phases slipped until one of the bounded waits ran out.
template <typename LT, typename GT, int A, int C, bool kPlain, bool kLong, int NT, bool kIndirect, int R>
__global__ void __launch_bounds__(C * (NT / R) + 32, 1)
impact_loss_categorical_ws_kernel(const __grid_constant__ CatParams p, const int S, const int W, const int lanes,
                                  const int n_prefetch) {
    constexpr int NP = (A + 1) / 2;
    constexpr int NTH = NT / R;  // threads of a consumer group: R steps of a tile each
    constexpr int WR = 32 * R;   // rows of a tile that one warp works on
    static_assert(R == 1 || (!kLong && A <= 32), "several steps per thread: trajectories within a tile, rows in registers");
    static_assert(NTH % 32 == 0 && NTH >= 32, "whole warps");
    constexpr bool kStream = (A > 32);
    static_assert(!kStream || (A % 2 == 0 && (NP & (NP - 1)) == 0), "streamed rows: an even, power-of-two pair count");
    constexpr int kInRow = A * (int)sizeof(LT), kOutRow = A * (int)sizeof(GT);
    constexpr int kInPitch = (int)ws_slab_pitch(NT, kInRow);
    constexpr int kStageBytes = (int)ws_stage_bytes<LT, GT, A, NT>();
    constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;
    using RM = RowMath<LT, A>;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kWsMaxStages], empty_bar[kWsMaxStages];
    __shared__ unsigned int tickets_s, tag_s;  // (see dev::draw_ticket_and_publish)
    __shared__ float2 warp_agg[C][2][NTH / 32];  // (two sets, used in turn: a tile's scan has one barrier)
    __shared__ __align__(16) float red[C][NTH / 32][8];
    __shared__ int abort_s;
    __shared__ float carry_s[C];

    const int tid = threadIdx.x, lane = tid & 31;
    const LossScalars& k = p.k;
    const TileGeometry& g = p.geo;
    const long long total_tiles = kLong ? g.nchunks * g.ntiles : g.nchunks;
    const int n_tiles = (int)((total_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x);  // this block's tiles
    const int rows_full = kLong ? NT : g.G * (int)g.T;                                   // rows of a full tile
    const long long total_rows = g.B * g.T;
    const long long agg_stride = g.tile_major ? 2 * g.B : 2;  // slots between a tile's aggregate and that of the tile after it in time
    auto place_of = [&](int n) { return tile_place<kLong, NT>(g, n, rows_full, total_rows); };
    // The tensors this launch reads: the call's own arguments (kernel parameters, read where they are used), or --
    // kIndirect: the call names a record in device memory that an earlier kernel of the stream fills (the circular
    // buffer's bookkeeping on the device) -- that record's, fetched once the stream dependency has resolved
    // (kept in shared memory, not in registers; the producer warp alone fetches the record, before the block-wide
    // barrier that releases the consumer warps: with every warp of the grid fetching it -- 3 000 warps asking one
    // cache line at the same moment -- the first tile was requested 3.6 us late)
    __shared__ LossInputPointers in_s;
#define IMPACT_IN(field) (kIndirect ? in_s.field : p.field)

    if (tid >= C * NTH) {
        // ---- producer warp ----------------------------------------------------------------------------------
        const int n_first = n_tiles < W ? n_tiles : W;
        // First of all, while the kernel before this one on the stream is still finishing, the warp asks L2 for
        // the block's first tiles (logits and per-step scalars), unless the launch's companion kernel has done so
        // already: the pages are mapped and the bytes on their way when the dependency resolves.
        if (n_prefetch > 0) {
            const void* base = nullptr;
            long long pitch = 4;
            if (lane == 0) { base = IMPACT_IN(learner_logits); pitch = kInRow; }
            else if (lane == 1) { base = IMPACT_IN(target_logits); pitch = kInRow; }
            else if (lane == 2) base = IMPACT_IN(actions);
            else if (lane == 3) base = IMPACT_IN(worker_logp);
            else if (lane == 4) base = IMPACT_IN(rewards);
            else if (lane == 5) base = IMPACT_IN(discounts);
            else if (lane == 6) base = IMPACT_IN(values);
            const int n_pf = n_tiles < n_prefetch ? n_tiles : n_prefetch;
            for (int n = 0; n < n_pf; ++n) {
                const Place pc = place_of(n);
                if (base) dev::prefetch_range_l2(base, pc.row0 * pitch, (uint32_t)(pc.nrows * pitch), total_rows * pitch);
            }
        }
        // then the barriers
        if (lane < S) {
            dev::mbarrier_init_nofence(&full_bar[lane], 1);
            dev::mbarrier_init_nofence(&empty_bar[lane], NTH / 32);  // one arrival per consumer warp
        }
        if (lane == 0) { abort_s = 0; tickets_s = 0u; }
        dev::fence_mbarrier_init();
        __syncwarp();

        // One slab of a tile into stage s: a bulk copy of the 16-byte granules that enclose the tile's rows
        // (dev::widen_range).  The lane with the learner's slab makes the barrier's one arrival, announcing the
        // bytes of both slabs; where the tensors end inside the last granule, it also fetches that granule's bytes
        // of both slabs by ordinary loads, fenced towards the copy engine because the consumers may send the target
        // rows on from the stage by a bulk store.
        const long long tensor_bytes = total_rows * kInRow;
        struct SlabRequest {
            unsigned char* d0;        // the learner's slab of the stage (the target's lies kInPitch further)
            const unsigned char* gl;  // first granule of the tile in the learner's logits
            const unsigned char* gt;  // ... in the target's
            uint32_t span, tail;      // dev::WideRange
        };
        auto request_for = [&](const Place& pc, int s) {
            const dev::WideRange w = dev::widen_range(pc.row0 * (long long)kInRow, (uint32_t)pc.nrows * kInRow, tensor_bytes);
            SlabRequest r;
            r.d0 = smem_raw + s * kStageBytes;  // the tile's first row starts (row0 * kInRow) mod 16 bytes in
            r.gl = static_cast<const unsigned char*>(IMPACT_IN(learner_logits)) + w.first;
            r.gt = static_cast<const unsigned char*>(IMPACT_IN(target_logits)) + w.first;
            r.span = w.span;
            r.tail = w.tail;
            return r;
        };
        auto send_slab = [&](const SlabRequest& r, int s, bool target) {
            uint64_t* const bar = &full_bar[s];
            if (target) {
                if (r.span) dev::bulk_load(r.d0 + kInPitch, r.gt, r.span, bar);
                return;
            }
            if (r.tail) {
                for (uint32_t i = 0; i < r.tail; ++i) {
                    r.d0[r.span + i] = r.gl[r.span + i];
                    r.d0[kInPitch + r.span + i] = r.gt[r.span + i];
                }
                dev::fence_async_shared();
            }
            if (r.span) {
                dev::mbarrier_expect_tx(bar, 2 * r.span);
                dev::bulk_load(r.d0, r.gl, r.span, bar);
            } else {
                dev::mbarrier_arrive(bar);
            }
        };
        // Tiles leave in rounds: lane l < 16 owns the round's l-th tile and requests its learner slab, lane l + 16
        // requests the same tile's target slab, so that all requests of a round leave in the same few instructions
        // (one thread gets at most four bulk requests under way, and needs about a third of a microsecond per
        // tile; a lane per request reaches the HBM rate).
        const int sub = lane & 15;
        const bool second = lane >= 16;
        // the first W tiles need no wait (tile n goes to stage n): their requests are worked out now and leave the
        // moment the stream's previous kernel is done, before the rest of the block has even started
        SlabRequest first = request_for(place_of(sub < n_first ? sub : 0), sub);

        grid_dependency_wait();

        if (kIndirect) {  // (the addresses were not known before)
            if (lane == 0) in_s = fetch_loss_inputs(p.indirect);
            __syncwarp();
            first = request_for(place_of(sub < n_first ? sub : 0), sub);
        }
        if (sub < n_first) send_slab(first, sub, second);
        __syncthreads();  // the barriers are set up: the consumer warps may use them
        const unsigned int tag = dev::launch_tag(p.counter);  // (asked for now, needed after the last tile has left)
        // The rest.  Tile n goes to stage n % S once that stage's previous tile has left (the "empty" phase before
        // this one) and tile n - W has landed (at most W tiles in flight).  The owners look at their barriers side by
        // side (one thread taking tile after tile through blocking waits costs a third of a microsecond per tile, too
        // much for small tiles: measured 33 us against 25 us on a million steps of six actions), but a tile is sent
        // only when every earlier tile of the round has been sent or is sent in the same instruction: tiles leave in
        // order.
        for (int base = n_first; base < n_tiles; base += lanes) {
            const int n = base + sub;
            bool pending = sub < lanes && n < n_tiles;
            const int cyc = n / S, s = n - cyc * S;
            const int wcyc = (n - W) / S, ws = (n - W) - wcyc * S;
            const SlabRequest req = request_for(place_of(pending ? n : 0), s);
            for (unsigned int spin = 0; spin < (1u << 22); ++spin) {
                const bool ready = !second && pending && (cyc == 0 || dev::mbarrier_test(&empty_bar[s], (uint32_t)(cyc - 1) & 1u)) &&
                                   dev::mbarrier_test(&full_bar[ws], (uint32_t)wcyc & 1u);
                const unsigned int waiting = __ballot_sync(0xffffffffu, !second && pending && !ready);
                bool go = ready && (waiting & ((1u << sub) - 1u)) == 0u;
                go = __shfl_sync(0xffffffffu, go, sub);  // the owner decides for both lanes of its tile
                if (go && pending) {
                    send_slab(req, s, second);
                    pending = false;
                }
                if (!__any_sync(0xffffffffu, pending)) break;
                if (*reinterpret_cast<volatile int*>(&abort_s)) break;
                __nanosleep(32);
            }
            if (__any_sync(0xffffffffu, pending)) {  // a stage never came back, or a tile never landed
                if (lane == 0) {
                    atomicExch(p.counter + 1, 1u);
                    *reinterpret_cast<volatile int*>(&abort_s) = 1;
                }
                break;
            }
        }
        __syncwarp();
        // ---- then it leaves this launch's tag for whoever publishes the block's sums, and draws its own ticket
        if (lane == 0) tag_s = tag;
        dev::draw_ticket_and_publish<C, NTH / 32>(&tickets_s, &tag_s, red, p.tagged_rows);
        return;
    }

    // ---- consumer groups ------------------------------------------------------------------
    // A group of NTH threads works on a tile of NT steps, R steps per thread: warp w of the group on the tile's
    // rows [WR w, WR (w + 1)), lane l of it on rows WR w + 32 i + l (i < R).  Everything a tile costs per thread
    // and not per step -- the waits, the placement, the hand-over of the stage, the stores' bookkeeping -- is paid
    // once for R steps, and a thread has R independent rows in flight.
    const int grp = tid / NTH, gtid = tid & (NTH - 1), gwarp = gtid >> 5;
    const int bar_id = grp + 1;
    const int wrow = gwarp * WR;  // the warp's first row in a tile
    const bool want_kl = !kPlain && (k.kl_coef != 0.0f);

    // (short trajectories) a thread's places in a tile never change: row tr[i] is step ts of trajectory q[i] of
    // the tile
    int tr[R], q[R];
    bool ends_short[R];
#pragma unroll
    for (int i = 0; i < R; ++i) {
        tr[i] = wrow + 32 * i + lane;
        q[i] = 0;
        int ts = tr[i];
        if (!kLong && g.G > 1) { q[i] = tr[i] / (int)g.T; ts = tr[i] - q[i] * (int)g.T; }
        ends_short[i] = ts == (int)g.T - 1;
    }
    // Where the group's next tile sits: short trajectories advance by a fixed number of rows and trajectories
    // (C tiles of the block further on), long ones are placed tile by tile.
    const long long group_row_stride = (long long)C * gridDim.x * rows_full;
    const long long group_traj_stride = (long long)C * gridDim.x * g.G;
    auto place_after = [&](const Place& pc, int n_next) {
        if constexpr (kLong) {
            return place_of(n_next < n_tiles ? n_next : 0);
        } else {
            Place pn;
            pn.row0 = pc.row0 + group_row_stride;
            pn.traj = pc.traj + group_traj_stride;
            const long long left = total_rows - pn.row0;
            pn.nrows = left < rows_full ? (left > 0 ? (int)left : 0) : rows_full;
            pn.r = 0;
            return pn;
        }
    };
    // does the thread's i-th row end its trajectory (in the tile at `pc`)?
    auto ends_trajectory = [&](const Place& pc, int i) {
        return kLong ? (pc.r == 0 && tr[i] == pc.nrows - 1) : ends_short[i];
    };

    struct StepRaw {
        int a;
        float l_worker, reward, discount, value, value_next;
    };
    // the per-step scalars of the thread's i-th row in the tile at `pc` (`has`: the block has such a tile)
    auto load_scalars = [&](const Place& pc, bool has, int i) {
        StepRaw x;
        x.a = 0; x.l_worker = 0.0f; x.reward = 0.0f; x.discount = 0.0f; x.value = 0.0f; x.value_next = 0.0f;
        if (has && tr[i] < pc.nrows) {
            // (loads that name the global space: a pointer taken from the device record is a generic one to the
            // compiler, and a generic load has to be complete before the next store to shared memory -- that put the
            // whole trip to L2 into every tile, 10.9 us a launch against 6.8)
            const long long r = pc.row0 + tr[i];
            const int a = __ldg(IMPACT_IN(actions) + r);
            x.a = min(max(a, 0), A - 1);
            x.l_worker = __ldg(IMPACT_IN(worker_logp) + r);
            x.reward = __ldg(IMPACT_IN(rewards) + r);
            x.discount = __ldg(IMPACT_IN(discounts) + r);
            x.value = __ldg(IMPACT_IN(values) + r);
            x.value_next = ends_trajectory(pc, i) ? __ldg(IMPACT_IN(bootstrap) + pc.traj + q[i]) : __ldg(IMPACT_IN(values) + r + 1);
        }
        return x;
    };

    float t_surr = 0.0f, t_val = 0.0f, t_ent = 0.0f, t_ratio = 0.0f, t_kl = 0.0f;
    int n_clip = 0, n_trunc = 0;
    // The group's sums, once final: a butterfly per warp into `red`, then the warp's ticket; the last ticket of
    // the block publishes its row (fixed order throughout).
    auto hand_over_sums = [&]() {
        dev::hand_over_warp_sums<C, NTH / 32>(t_surr, t_val, t_ent, t_ratio, t_kl, want_kl,
                                              __reduce_add_sync(0xffffffffu, n_clip), __reduce_add_sync(0xffffffffu, n_trunc),
                                              red[grp][gwarp], &tickets_s, &tag_s, red, p.tagged_rows);
    };

    bool pending = false;  // lane 0 of each warp: a store of this warp may still be reading its stage
    int pending_stage = 0;

    grid_dependency_wait();
    Place pc = place_of(grp < n_tiles ? grp : 0);
    StepRaw cur[R];
    if (!kIndirect) {
#pragma unroll
        for (int i = 0; i < R; ++i) cur[i] = load_scalars(pc, grp < n_tiles, i);
    }
    __syncthreads();  // the producer warp has set up the barriers (and fetched the device record)
    if (kIndirect) {
#pragma unroll
        for (int i = 0; i < R; ++i) cur[i] = load_scalars(pc, grp < n_tiles, i);
    }
    int s = grp % S;
    uint32_t ph = (uint32_t)(grp / S) & 1u;
    int turn = 0;  // which of the group's two sets of warp aggregates this tile uses

    for (int n = grp; n < n_tiles; n += C) {
        // the next tile's scalars travel while this tile is worked on
        const Place pc_next = place_after(pc, n + C);
        StepRaw nxt[R];
#pragma unroll
        for (int i = 0; i < R; ++i) nxt[i] = load_scalars(pc_next, n + C < n_tiles, i);
        // this warp's previous rows have left shared memory: hand the stage back.  (Only where stages are used
        // more than once: the wait for the store's reads sits between two tiles of the warp, and a block with no
        // more tiles than stages never needs a stage back.)
        if (lane == 0 && pending) {
            dev::bulk_store_wait_read();
            dev::mbarrier_arrive(&empty_bar[pending_stage]);
            pending = false;
        }
        // every thread waits for the stage itself (a bounded wait: on a time-out the flag is set and the
        // thread goes on with whatever the stage holds, so that all barriers below still pair up)
        // (long trajectories) one early look at the aggregates of the later tiles of this tile's trajectory: with
        // many trajectories they were published a round ago, and reading them now keeps that trip to L2 off the
        // path between this tile's scan and its gradients
        // (only where tiles are numbered tile-major; the values are first looked at after the scan)
        const bool peeked = kLong && g.tile_major && gwarp == 0 && pc.r > lane;
        unsigned long long early_a = 0, early_b = 0;
        if (peeked)
            dev::load_aggregate(p.tile_aggregates + 2 * ((long long)blockIdx.x + (long long)n * gridDim.x), agg_stride,
                                pc.r - lane, early_a, early_b);
        if (!dev::mbarrier_wait(&full_bar[s], ph, &abort_s)) atomicExch(p.counter + 1, 1u);

        // rows keep their place inside their 16-byte granule: the tile's first row starts (row0 * pitch) mod 16
        // bytes into the slab
        unsigned char* const stage = smem_raw + s * kStageBytes;
        const uint32_t m_in = (uint32_t)(pc.row0 * kInRow) & 15u;
        unsigned char* const s0 = stage + m_in;     // learner logits
        unsigned char* const s1 = s0 + kInPitch;    // target logits
        unsigned char* const so = (sizeof(LT) == sizeof(GT)) ? s0 : stage + 2 * kInPitch + ((uint32_t)(pc.row0 * kOutRow) & 15u);
        bool stored = false;  // lane 0: a bulk store of this warp reads the stage
        // the warp's rows of this tile
        const int wleft = pc.nrows - wrow;
        const int wrows = wleft > WR ? WR : (wleft > 0 ? wleft : 0);
        const long long wrow0 = pc.row0 + wrow;
        // (first traversal of a batch) the target rows go to the circular buffer as well, each warp's rows
        // straight from the stage, which nothing writes to
        if (IMPACT_IN(target_copy)) {
            unsigned char* const dst = static_cast<unsigned char*>(IMPACT_IN(target_copy)) + wrow0 * (long long)kInRow;
            stored = dev::warp_send_bytes(dst, s1 + wrow * kInRow, (uint32_t)wrows * kInRow, false);
        }

        // ---- row passes (every thread; rows beyond the tile hold stale bytes and are masked)
        dev::StepIn st[R];
        float2 e[R][kStream ? 1 : NP];
        float lse2_t[R], lse2_l[R], inv_s[R], ent[R], m2_l[R], kl[R];
        float fa[R], fb[R];
        bool active[R], truncated[R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int row = tr[i];
            active[i] = row < pc.nrows;
            st[i].l_worker = cur[i].l_worker;
            st[i].reward = cur[i].reward;
            st[i].discount = cur[i].discount;
            st[i].value = cur[i].value;
            st[i].value_next = cur[i].value_next;
            st[i].last_step = ends_trajectory(pc, i);
            m2_l[i] = 0.0f;
            kl[i] = 0.0f;
            if constexpr (!kStream) {
                float m2_t, sum_t, unused, sum_l, sez;
                lse2_t[i] = RM::template lse2<false>(s1, row, e[i], m2_t, sum_t, unused);
                lse2_l[i] = RM::template lse2<true>(s0, row, e[i], m2_l[i], sum_l, sez);
                inv_s[i] = dev::rcp_fast(sum_l);
                // H = -sum_j pi_j lp_j = (m + ln S) - sum_j e_j z_j / S
                ent[i] = fmaf(lse2_l[i], kLn2, -sez * inv_s[i]);
                if (want_kl) {
#pragma unroll
                    for (int j = 0; j < A; ++j) {
                        const float lpt2 = fmaf(RowIO<LT, A>::at(s1, row, j), kLog2e, -lse2_t[i]);
                        const float lpl2 = fmaf(RowIO<LT, A>::at(s0, row, j), kLog2e, -lse2_l[i]);
                        kl[i] = fmaf(dev::exp2_fast(lpt2), (lpt2 - lpl2) * kLn2, kl[i]);
                    }
                }
            } else {
                const int skew = row & (NP - 1);
                const float2 log2e2 = make_float2(kLog2e, kLog2e);
                auto row_max2 = [&](const unsigned char* slab) {
                    float2 mx = RowIO<LT, A>::load_pair(slab, row, skew);
#pragma unroll 8
                    for (int j = 1; j < NP; ++j) {
                        const float2 v = RowIO<LT, A>::load_pair(slab, row, (j + skew) & (NP - 1));
                        mx.x = fmaxf(mx.x, v.x);
                        mx.y = fmaxf(mx.y, v.y);
                    }
                    return fmaxf(mx.x, mx.y) * kLog2e;
                };
                {   // target row: its log-sum-exp
                    const float m2 = row_max2(s1);
                    const float2 neg_m2 = make_float2(-m2, -m2);
                    float2 sum2 = make_float2(0.0f, 0.0f);
#pragma unroll 8
                    for (int j = 0; j < NP; ++j) {
                        const float2 t2 = __ffma2_rn(RowIO<LT, A>::load_pair(s1, row, (j + skew) & (NP - 1)), log2e2, neg_m2);
                        sum2 = __fadd2_rn(sum2, make_float2(dev::exp2_fast(t2.x), dev::exp2_fast(t2.y)));
                    }
                    lse2_t[i] = m2 + dev::log2_fast(sum2.x + sum2.y);
                }
                {   // learner row: log-sum-exp and sum_j e_j z_j
                    m2_l[i] = row_max2(s0);
                    const float2 neg_m2 = make_float2(-m2_l[i], -m2_l[i]);
                    float2 sum2 = make_float2(0.0f, 0.0f), sez2 = make_float2(0.0f, 0.0f);
#pragma unroll 8
                    for (int j = 0; j < NP; ++j) {
                        const float2 z = RowIO<LT, A>::load_pair(s0, row, (j + skew) & (NP - 1));
                        const float2 t2 = __ffma2_rn(z, log2e2, neg_m2);
                        const float2 ex = make_float2(dev::exp2_fast(t2.x), dev::exp2_fast(t2.y));
                        sum2 = __fadd2_rn(sum2, ex);
                        sez2 = __ffma2_rn(ex, z, sez2);
                    }
                    const float sum_l = sum2.x + sum2.y;
                    lse2_l[i] = m2_l[i] + dev::log2_fast(sum_l);
                    inv_s[i] = dev::rcp_fast(sum_l);
                    ent[i] = fmaf(lse2_l[i], kLn2, -(sez2.x + sez2.y) * inv_s[i]);
                }
                if (want_kl) {
#pragma unroll 8
                    for (int j = 0; j < NP; ++j) {
                        const int jj = (j + skew) & (NP - 1);
                        const float2 zt2 = RowIO<LT, A>::load_pair(s1, row, jj), zl2 = RowIO<LT, A>::load_pair(s0, row, jj);
                        const float ax = fmaf(zt2.x, kLog2e, -lse2_t[i]), ay = fmaf(zt2.y, kLog2e, -lse2_t[i]);
                        kl[i] = fmaf(dev::exp2_fast(ax), (ax - fmaf(zl2.x, kLog2e, -lse2_l[i])) * kLn2, kl[i]);
                        kl[i] = fmaf(dev::exp2_fast(ay), (ay - fmaf(zl2.y, kLog2e, -lse2_l[i])) * kLn2, kl[i]);
                    }
                }
            }
            st[i].l_target = fmaf(RowIO<LT, A>::at(s1, row, cur[i].a), kLog2e, -lse2_t[i]) * kLn2;
            st[i].l_theta = fmaf(RowIO<LT, A>::at(s0, row, cur[i].a), kLog2e, -lse2_l[i]) * kLn2;
            if (kPlain) truncated[i] = dev::recursion_map_plain(st[i], k, fa[i], fb[i]);
            else truncated[i] = dev::recursion_map(st[i], k, fa[i], fb[i]);
            if (!active[i]) { fa[i] = 1.0f; fb[i] = 0.0f; }
        }
        float adv[R];
        if constexpr (!kLong) {
            float adv_next[R];
            dev::suffix_affine_scan_rows<NTH, R>(fa, fb, warp_agg[grp][turn], adv, adv_next, bar_id);
#pragma unroll
            for (int i = 0; i < R; ++i) st[i].adv_next = adv_next[i];
        } else {
            // maps instead of values: (ma, mb) takes the value that enters the tile's last step to A of this
            // step, (la, lb) to A of the step after this warp's last
            float ma, mb, la, lb;
            dev::suffix_affine_maps_group<NT>(fa[0], fb[0], warp_agg[grp][turn], ma, mb, la, lb, bar_id);
            const long long gtile = (long long)blockIdx.x + (long long)n * gridDim.x;
            if (gtid == 0) dev::publish_tile_aggregate(p.tile_aggregates + 2 * gtile, ma, mb, dev::launch_tag(p.counter));
            float carry = 0.0f;
            if (pc.r > 0) {  // uniform over the group
                if (gwarp == 0) {
                    const float c = dev::compose_later_aggregates(p.tile_aggregates + 2 * gtile, agg_stride, pc.r,
                                                                  dev::launch_tag(p.counter), &abort_s, peeked,
                                                                  early_a, early_b);
                    if (lane == 0) carry_s[grp] = c;
                }
                asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(NT) : "memory");
                carry = carry_s[grp];
            }
            adv[0] = fmaf(ma, carry, mb);
            const float below = __shfl_down_sync(0xffffffffu, adv[0], 1);
            st[0].adv_next = (lane == 31) ? fmaf(la, carry, lb) : below;
        }
        turn ^= 1;

        float wpg[R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            float surr, ratio;
            bool clipped;
            wpg[i] = kPlain ? dev::surrogate_plain(st[i], k, adv[i], surr, ratio, clipped)
                            : dev::surrogate(st[i], k, adv[i], surr, ratio, clipped);
            if (active[i]) {
                t_surr += surr;
                t_val = fmaf(0.5f * adv[i], adv[i], t_val);
                t_ent += ent[i];
                t_ratio += ratio;
                if (!kPlain) t_kl += kl[i];
            }
            n_clip += (active[i] && clipped) ? 1 : 0;  // (per thread; added up over the warp when the sums are handed over)
            n_trunc += (active[i] && truncated[i]) ? 1 : 0;
        }
        // the group's sums are final after its last tile's scan: handed over here, they are published while
        // that tile's gradient pass runs
        if (n + C >= n_tiles) hand_over_sums();

        // ---- gradients: row_j = e_j (ga z_j + gb) [- kl_coef pi_target_j / M], then the taken action's entry
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int row = tr[i];
            const float w1 = wpg[i] * k.inv_M, ce = k.ent_coef * k.inv_M, ck = kPlain ? 0.0f : k.kl_coef * k.inv_M;
            const float h_off = fmaf(-lse2_l[i], kLn2, ent[i]);
            const float ga = ce * inv_s[i], gb = (fmaf(ce, h_off, w1) + ck) * inv_s[i];
            const float2 ga2 = make_float2(ga, ga), gb2 = make_float2(gb, gb);
            if constexpr (!kStream) {
                if (!want_kl) {
#pragma unroll
                    for (int j = 0; j < NP; ++j) {
                        const float2 z = RowIO<LT, A>::load_pair(s0, row, j);
                        RowIO<GT, A>::store_pair(so, row, j, __fmul2_rn(e[i][j], __ffma2_rn(z, ga2, gb2)));
                    }
                } else {
                    const float2 neg_lse2 = make_float2(-lse2_t[i], -lse2_t[i]), nck2 = make_float2(-ck, -ck);
                    const float2 log2e2 = make_float2(kLog2e, kLog2e);
#pragma unroll
                    for (int j = 0; j < NP; ++j) {
                        const float2 z = RowIO<LT, A>::load_pair(s0, row, j);
                        const float2 tt = __ffma2_rn(RowIO<LT, A>::load_pair(s1, row, j), log2e2, neg_lse2);
                        const float2 pt = make_float2(dev::exp2_fast(tt.x), dev::exp2_fast(tt.y));
                        RowIO<GT, A>::store_pair(so, row, j, __ffma2_rn(nck2, pt, __fmul2_rn(e[i][j], __ffma2_rn(z, ga2, gb2))));
                    }
                }
            } else {
                const int skew = row & (NP - 1);
                const float2 log2e2 = make_float2(kLog2e, kLog2e), neg_m2 = make_float2(-m2_l[i], -m2_l[i]);
                const float2 neg_lse2 = make_float2(-lse2_t[i], -lse2_t[i]), nck2 = make_float2(-ck, -ck);
#pragma unroll 8
                for (int j = 0; j < NP; ++j) {
                    const int jj = (j + skew) & (NP - 1);
                    const float2 z = RowIO<LT, A>::load_pair(s0, row, jj);
                    const float2 t2 = __ffma2_rn(z, log2e2, neg_m2);
                    const float2 ex = make_float2(dev::exp2_fast(t2.x), dev::exp2_fast(t2.y));
                    float2 gr = __fmul2_rn(ex, __ffma2_rn(z, ga2, gb2));
                    if (want_kl) {
                        const float2 tt = __ffma2_rn(RowIO<LT, A>::load_pair(s1, row, jj), log2e2, neg_lse2);
                        gr = __ffma2_rn(nck2, make_float2(dev::exp2_fast(tt.x), dev::exp2_fast(tt.y)), gr);
                    }
                    RowIO<GT, A>::store_pair(so, row, jj, gr);
                }
            }
            const float pi_a = dev::exp2_fast(st[i].l_theta * kLog2e);
            float g_a = fmaf(pi_a, fmaf(ce, st[i].l_theta + ent[i], w1), -w1);
            if (want_kl) g_a = fmaf(ck, pi_a - dev::exp2_fast(st[i].l_target * kLog2e), g_a);
            if (active[i]) {
                const long long grow = pc.row0 + row;
                p.dvalues[grow] = -k.vf_coef * k.inv_M * adv[i];  // V - Vhat = -A
                if (!kPlain) {
                    if (p.vtarget) p.vtarget[grow] = st[i].value + adv[i];
                    if (p.advantage) p.advantage[grow] = adv[i];
                }
            }
            RowIO<GT, A>::put(so, row, cur[i].a, g_a);
        }
        // ---- each warp sends its own rows: no barrier across the group
        {
            unsigned char* const gd = static_cast<unsigned char*>(p.dlogits) + wrow0 * (long long)kOutRow;
            if (dev::warp_send_bytes(gd, so + wrow * kOutRow, (uint32_t)wrows * kOutRow, true)) stored = true;
            if (lane == 0) {
                if (stored) {  // the stage goes back once the stores have read it: before this warp's next tile
                    pending = n_tiles > S;
                    pending_stage = s;
                } else {
                    dev::mbarrier_arrive(&empty_bar[s]);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < R; ++i) cur[i] = nxt[i];
        pc = pc_next;
        s += C;
        while (s >= S) { s -= S; ph ^= 1u; }
    }

    // a group without tiles still hands over its (zero) sums, so that every row of the grid is defined
    if (grp >= n_tiles) hand_over_sums();
    // ---- one group of the grid (block 0's, the one that runs out of tiles first and so is polling long before the
    // last rows appear) collects every block's row
    // as it appears and writes the loss terms
    if (blockIdx.x == 0 && grp == n_tiles % C) {
        if (!dev::reduce_tagged_rows<NTH>(p.tagged_rows, (int)gridDim.x, dev::launch_tag(p.counter), p.counter,
                                          p.loss_terms, k.vf_coef, k.ent_coef, k.kl_coef, k.steps_total,
                                          gtid, bar_id, &abort_s))
            if (gtid == 0) atomicExch(p.counter + 1, 1u);
    }
    if (lane == 0) dev::bulk_store_wait_read();  // shared memory must outlive the stores' reads
#undef IMPACT_IN
}

// ------------------------------------------------------------------------------------------
// Diagonal-Gaussian policy
// ------------------------------------------------------------------------------------------
template <int NT>
__global__ void __launch_bounds__(NT) impact_loss_gaussian_kernel(const GaussParams p) {
    grid_dependency_wait();
    extern __shared__ __align__(16) float smem[];
    const int D = p.D, Ds = p.Ds;
    float* const s_mu = smem;                              // learner mean -> dmean
    float* const s_ls = s_mu + (size_t)NT * Ds;            // learner logstd -> dlogstd
    float* const s_mt = s_ls + (size_t)NT * Ds;            // target mean
    float* const s_lt = s_mt + (size_t)NT * Ds;            // target logstd
    float* const s_ac = s_lt + (size_t)NT * Ds;            // actions
    __shared__ float2 warp_agg[NT / 32];
    __shared__ float red[NT / 32][8];
    __shared__ float carry_s;

    const int tid = threadIdx.x;
    const LossScalars k = p.k;
    const TileGeometry g = p.geo;
    const float half_log_2pi = 0.91893853320467274178f;

    float acc[dev::kNumSums];
#pragma unroll
    for (int j = 0; j < dev::kNumSums; ++j) acc[j] = 0.0f;

    for (long long chunk = blockIdx.x; chunk < g.nchunks; chunk += gridDim.x) {
        float carry = 0.0f;
        for (int tile = g.ntiles - 1; tile >= 0; --tile) {
            const TileRows tr = tile_rows<NT>(g, chunk, tile);
            const long long base = tr.row0 * D;
            const int nelem = tr.nrows * D;
            __syncthreads();
            dev::stage_slab<float, NT>(s_mu, p.learner_mean, base, nelem, D, Ds);
            dev::stage_slab<float, NT>(s_ls, p.learner_logstd, base, nelem, D, Ds);
            dev::stage_slab<float, NT>(s_mt, p.target_mean, base, nelem, D, Ds);
            dev::stage_slab<float, NT>(s_lt, p.target_logstd, base, nelem, D, Ds);
            dev::stage_slab<float, NT>(s_ac, p.actions, base, nelem, D, Ds);
            __syncthreads();

            const bool active = tid < tr.nrows;
            const long long row = tr.row0 + tid;
            float* const r_mu = s_mu + tid * Ds;
            float* const r_ls = s_ls + tid * Ds;
            const float* const r_mt = s_mt + tid * Ds;
            const float* const r_lt = s_lt + tid * Ds;
            const float* const r_ac = s_ac + tid * Ds;
            dev::StepIn s;
            float fa = 1.0f, fb = 0.0f;
            float ent = 0.0f, kl = 0.0f;
            bool truncated = false;
            if (active) {
                long long b, t;
                if (g.ntiles > 1) { b = chunk; t = (long long)tile * NT + tid; }
                else { const int q = tid / (int)g.T; b = chunk * g.G + q; t = tid - q * (int)g.T; }
                // The log-probabilities are sums of D terms and reach magnitudes of tens; they
                // enter exponentials, so their absolute error is the relative error of the
                // ratios.  Accumulating them in fp64 (half-rate on this part, a few percent of
                // the pipe here) keeps that error at the level of the fp32 terms themselves.
                double lth = 0.0, ltg = 0.0;
                for (int j = 0; j < D; ++j) {
                    const float ls = r_ls[j], lt = r_lt[j], ac = r_ac[j];
                    const float inv_s = expf(-ls), inv_st = expf(-lt);
                    const float z1 = (ac - r_mu[j]) * inv_s;
                    const float z2 = (ac - r_mt[j]) * inv_st;
                    lth += (double)(fmaf(-0.5f * z1, z1, -ls) - half_log_2pi);
                    ltg += (double)(fmaf(-0.5f * z2, z2, -lt) - half_log_2pi);
                    ent += ls + (half_log_2pi + 0.5f);
                    if (k.kl_coef != 0.0f) {  // KL(target || learner), per dimension
                        const float dm = (r_mt[j] - r_mu[j]) * inv_s;
                        const float sr = expf(lt - ls);  // sigma_target / sigma_learner
                        kl += (ls - lt) + 0.5f * fmaf(sr, sr, dm * dm) - 0.5f;
                    }
                }
                // differences against the worker's log-probability are taken in fp64, then
                // everything continues in fp32 relative to it
                const float lw = p.worker_logp[row];
                s.l_theta = (float)(lth - (double)lw);
                s.l_target = (float)(ltg - (double)lw);
                s.l_worker = 0.0f;
                s.l_shift = lw;
                s.reward = p.rewards[row];
                s.discount = p.discounts[row];
                s.value = p.values[row];
                s.last_step = (t == g.T - 1);
                s.value_next = s.last_step ? p.bootstrap[b] : p.values[row + 1];
                asm volatile("" ::: "memory");
                truncated = dev::recursion_map(s, k, fa, fb);
            }
            const float adv = dev::suffix_affine_scan<NT>(fa, fb, carry, warp_agg, s.adv_next);
            if (tid == 0) carry_s = adv;

            float sums[dev::kNumSums];
#pragma unroll
            for (int j = 0; j < dev::kNumSums; ++j) sums[j] = 0.0f;
            if (active) {
                float surr, ratio;
                bool clipped;
                const float wpg = dev::surrogate(s, k, adv, surr, ratio, clipped);
                const float w1 = wpg * k.inv_M, ce = k.ent_coef * k.inv_M, ck = k.kl_coef * k.inv_M;
                for (int j = 0; j < D; ++j) {
                    const float ls = r_ls[j], lt = r_lt[j], mu = r_mu[j];
                    const float inv_s = expf(-ls);
                    const float z = (r_ac[j] - mu) * inv_s;       // (a - mu) / sigma
                    const float dm = (mu - r_mt[j]) * inv_s;      // (mu - mu_target) / sigma
                    const float sr = expf(lt - ls);
                    // d log pi / d mu = z / sigma ; d KL / d mu = dm / sigma
                    r_mu[j] = (ck * dm - w1 * z) * inv_s;
                    // d log pi / d logstd = z^2 - 1 ; d H / d logstd = 1 ;
                    // d KL / d logstd = 1 - (sigma_t^2 + (mu_t - mu)^2) / sigma^2
                    r_ls[j] = -w1 * fmaf(z, z, -1.0f) - ce + ck * (1.0f - fmaf(sr, sr, dm * dm));
                }
                p.dvalues[row] = -k.vf_coef * k.inv_M * adv;
                if (p.vtarget) p.vtarget[row] = s.value + adv;
                if (p.advantage) p.advantage[row] = adv;
                sums[0] = surr;
                sums[1] = 0.5f * adv * adv;
                sums[2] = ent;
                sums[3] = kl;
                sums[4] = clipped ? 1.0f : 0.0f;
                sums[5] = truncated ? 1.0f : 0.0f;
                sums[6] = ratio;
            }
            dev::block_sums_stage1<NT>(sums, red);
            __syncthreads();
            carry = carry_s;
            dev::unstage_slab<float, NT>(p.dmean, s_mu, base, nelem, D, Ds);
            dev::unstage_slab<float, NT>(p.dlogstd, s_ls, base, nelem, D, Ds);
            dev::block_sums_stage2<NT>(acc, red);
        }
    }
    dev::finish_loss_terms<NT>(acc, p.partials, p.counter, p.loss_terms, k,
                               k.steps_total);
}

// ------------------------------------------------------------------------------------------
// Diagonal-Gaussian policy, action dimension known at compile time
// ------------------------------------------------------------------------------------------
// Same structure as the register-resident categorical kernel: the five [tile, D] slabs
// (learner mean / log-std, target mean / log-std, actions) arrive by bulk copies, a thread
// walks its row with every loop unrolled, dmean / dlogstd replace the learner slabs in place and
// leave by two bulk stores.  One stage per block (five slabs are 43 KB at D = 17), four
// blocks per SM overlap each other's loads and arithmetic.
template <int D>
__global__ void __launch_bounds__(kRegTileRows, 4) impact_loss_gaussian_reg_kernel(const GaussParams p) {
    grid_dependency_wait();
    constexpr int NT = kRegTileRows;
    constexpr int kSlab = NT * D * (int)sizeof(float);
    constexpr float kLog2e = 1.4426950408889634f;
    constexpr float kHalfLog2Pi = 0.91893853320467274178f;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float* const s_mu = reinterpret_cast<float*>(smem_raw);              // learner mean -> dmean
    float* const s_ls = reinterpret_cast<float*>(smem_raw + kSlab);      // learner log-std -> dlogstd
    const float* const s_mt = reinterpret_cast<const float*>(smem_raw + 2 * kSlab);
    const float* const s_lt = reinterpret_cast<const float*>(smem_raw + 3 * kSlab);
    const float* const s_ac = reinterpret_cast<const float*>(smem_raw + 4 * kSlab);
    __shared__ __align__(8) uint64_t bar;
    __shared__ float2 warp_agg[NT / 32];
    __shared__ float red[NT / 32][8];
    __shared__ float carry_s;
    __shared__ int is_last_s;

    const int tid = threadIdx.x;
    const LossScalars k = p.k;
    const TileGeometry g = p.geo;
    const bool want_kl = (k.kl_coef != 0.0f);
    const float* const src[5] = {p.learner_mean, p.learner_logstd, p.target_mean, p.target_logstd, p.actions};

    if (tid == 0) {
        dev::mbarrier_init(&bar, 1);
        is_last_s = 0;
    }
    __syncthreads();
    uint32_t parity = 0;

    float acc[dev::kNumSums], tsum[dev::kNumSums];
#pragma unroll
    for (int j = 0; j < dev::kNumSums; ++j) acc[j] = tsum[j] = 0.0f;

    for (long long chunk = blockIdx.x; chunk < g.nchunks; chunk += gridDim.x) {
        float carry = 0.0f;
        for (int tile = g.ntiles - 1; tile >= 0; --tile) {
            const bool final_tile = (tile == 0) && (chunk + gridDim.x >= g.nchunks);
            const TileRows tr = tile_rows<NT>(g, chunk, tile);
            const long long base = tr.row0 * D;
            const uint32_t bytes = (uint32_t)tr.nrows * D * (uint32_t)sizeof(float);
            uintptr_t align = bytes;
#pragma unroll
            for (int q = 0; q < 5; ++q) align |= reinterpret_cast<uintptr_t>(src[q] + base);
            const bool bulk_in = (align & 15u) == 0;
            const bool bulk_out = (((reinterpret_cast<uintptr_t>(p.dmean + base) |
                                     reinterpret_cast<uintptr_t>(p.dlogstd + base) | bytes) & 15u) == 0);
            if (bulk_in) {
                if (tid == 0) {
                    dev::mbarrier_expect_tx(&bar, 5 * bytes);
#pragma unroll
                    for (int q = 0; q < 5; ++q) dev::bulk_load(smem_raw + q * kSlab, src[q] + base, bytes, &bar);
                }
            } else {
                const int nelem = tr.nrows * D;
#pragma unroll
                for (int q = 0; q < 5; ++q)
                    for (int e = tid; e < nelem; e += NT) reinterpret_cast<float*>(smem_raw + q * kSlab)[e] = src[q][base + e];
            }

            const bool active = tid < tr.nrows;
            const long long row = tr.row0 + tid;
            dev::StepIn s;
            float lw = 0.0f;
            if (active) {
                long long b, t;
                if (g.ntiles > 1) { b = chunk; t = (long long)tile * NT + tid; }
                else if (g.G == 1) { b = chunk; t = tid; }
                else { const int q = tid / (int)g.T; b = chunk * g.G + q; t = tid - q * (int)g.T; }
                lw = p.worker_logp[row];
                s.reward = p.rewards[row];
                s.discount = p.discounts[row];
                s.value = p.values[row];
                s.last_step = (t == g.T - 1);
                s.value_next = s.last_step ? p.bootstrap[b] : p.values[row + 1];
            }
            if (bulk_in) {
                if (tid < 32) {
                    if (!dev::mbarrier_wait(&bar, parity)) atomicExch(p.counter + 1, 1u);
                }
                parity ^= 1u;
            }
            __syncthreads();

            float* const r_mu = s_mu + tid * D;
            float* const r_ls = s_ls + tid * D;
            const float* const r_mt = s_mt + tid * D;
            const float* const r_lt = s_lt + tid * D;
            const float* const r_ac = s_ac + tid * D;
            float fa = 1.0f, fb = 0.0f, ent = 0.0f, kl = 0.0f;
            bool truncated = false;
            if (active) {
                // log-probabilities: D-term sums of magnitude tens that end up in exponents, so they
                // are accumulated in fp64 (half-rate here, a few percent of the pipe)
                double lth = 0.0, ltg = 0.0;
                float ls_sum = 0.0f;
#pragma unroll
                for (int j = 0; j < D; ++j) {
                    const float ls = r_ls[j], lt = r_lt[j], ac = r_ac[j], mu = r_mu[j], mt = r_mt[j];
                    const float inv_s = dev::exp2_fast(-ls * kLog2e), inv_st = dev::exp2_fast(-lt * kLog2e);
                    const float z1 = (ac - mu) * inv_s;
                    const float z2 = (ac - mt) * inv_st;
                    lth += (double)fmaf(-0.5f * z1, z1, -ls);
                    ltg += (double)fmaf(-0.5f * z2, z2, -lt);
                    ls_sum += ls;
                    if (want_kl) {  // KL(target || learner), per dimension
                        const float dm = (mt - mu) * inv_s;
                        const float sr = dev::exp2_fast((lt - ls) * kLog2e);  // sigma_target / sigma_learner
                        kl += (ls - lt) + 0.5f * fmaf(sr, sr, dm * dm) - 0.5f;
                    }
                }
                ent = ls_sum + (float)D * (kHalfLog2Pi + 0.5f);
                const double shift = (double)lw + (double)D * (double)kHalfLog2Pi;
                // everything downstream works on log-probabilities relative to the worker's
                s.l_theta = (float)(lth - shift);
                s.l_target = (float)(ltg - shift);
                s.l_worker = 0.0f;
                s.l_shift = lw;
                truncated = dev::recursion_map(s, k, fa, fb);
            }
            const float adv = dev::suffix_affine_scan<NT>(fa, fb, carry, warp_agg, s.adv_next);
            if (tid == 0) carry_s = adv;

            float surr = 0.0f, ratio = 0.0f, wpg = 0.0f;
            bool clipped = false;
            if (active) wpg = dev::surrogate(s, k, adv, surr, ratio, clipped);
            // each thread keeps its own running sums over the block's tiles; they are added across
            // the block once, in the last tile, and published right away so that the round trip
            // hides behind the epilogue
            if (active) {
                tsum[0] += surr;
                tsum[1] = fmaf(0.5f * adv, adv, tsum[1]);
                tsum[2] += ent;
                tsum[3] += kl;
                tsum[4] += clipped ? 1.0f : 0.0f;
                tsum[5] += truncated ? 1.0f : 0.0f;
                tsum[6] += ratio;
            }
            unsigned int ticket = 0;
            if (final_tile) {
                dev::block_sums_stage1<NT>(tsum, red);
                __syncthreads();
                if (tid == 0) {
                    dev::block_sums_stage2<NT>(acc, red);
                    ticket = dev::publish_block_sums(acc, p.partials, p.counter);
                }
            }
            if (active) {
                const float w1 = wpg * k.inv_M, ce = k.ent_coef * k.inv_M, ck = k.kl_coef * k.inv_M;
#pragma unroll
                for (int j = 0; j < D; ++j) {
                    const float ls = r_ls[j], mu = r_mu[j];
                    const float inv_s = dev::exp2_fast(-ls * kLog2e);
                    const float z = (r_ac[j] - mu) * inv_s;  // (a - mu) / sigma
                    // d log pi / d mu = z / sigma ;  d log pi / d logstd = z^2 - 1 ;  d H / d logstd = 1
                    float gm = -w1 * z;
                    float gs = -w1 * fmaf(z, z, -1.0f) - ce;
                    if (want_kl) {
                        // d KL / d mu = (mu - mu_t) / sigma^2 ; d KL / d logstd = 1 - (sigma_t^2 + (mu_t - mu)^2) / sigma^2
                        const float dm = (mu - r_mt[j]) * inv_s;
                        const float sr = dev::exp2_fast((r_lt[j] - ls) * kLog2e);
                        gm = fmaf(ck, dm, gm);
                        gs = fmaf(ck, 1.0f - fmaf(sr, sr, dm * dm), gs);
                    }
                    r_mu[j] = gm * inv_s;
                    r_ls[j] = gs;
                }
                p.dvalues[row] = -k.vf_coef * k.inv_M * adv;
                if (p.vtarget) p.vtarget[row] = s.value + adv;
                if (p.advantage) p.advantage[row] = adv;
            }
            if (bulk_out) dev::fence_async_shared();
            if (tid == 0 && final_tile) is_last_s = (ticket == gridDim.x - 1) ? 1 : 0;
            __syncthreads();
            carry = carry_s;
            if (bulk_out) {
                if (tid == 0) {
                    dev::bulk_store(p.dmean + base, s_mu, bytes);
                    dev::bulk_store(p.dlogstd + base, s_ls, bytes);
                    if (!final_tile) dev::bulk_store_wait_read();
                }
            } else {
                const int nelem = tr.nrows * D;
                for (int i = tid; i < nelem; i += NT) {
                    p.dmean[base + i] = s_mu[i];
                    p.dlogstd[base + i] = s_ls[i];
                }
            }
            if (!final_tile) __syncthreads();
        }
    }
    if (is_last_s) dev::reduce_published_sums<NT>(p.partials, p.counter, p.loss_terms, k.vf_coef, k.ent_coef, k.kl_coef,
                                                   k.steps_total);
    if (tid == 0) dev::bulk_store_wait_read();
}

// ------------------------------------------------------------------------------------------
// Diagonal-Gaussian policy, persistent warp-specialised form (trajectories of at most 128 steps)
// ------------------------------------------------------------------------------------------
// The structure of impact_loss_categorical_ws_kernel with five input slabs per tile (learner mean /
// log-std, target mean / log-std, actions) and two output slabs (dmean, dlogstd, written over the
// learner's): a producer warp streams tiles through the ring, C consumer groups take them as they
// land, every warp stores its own rows, the block's sums leave as one tagged row.  Row arithmetic is
// that of impact_loss_gaussian_reg_kernel (log-probabilities accumulated in fp64).  kLong as in the
// categorical kernel: tiles of a long trajectory on neighbouring blocks, linked through their aggregates.
template <int D>
__host__ __device__ constexpr size_t gaussian_ws_stage_bytes() {
    return (5 * ws_slab_pitch(128, D * sizeof(float)) + 127) / 128 * 128;
}

template <int D, int C, bool kLong>
__global__ void __launch_bounds__(C * 128 + 32, 1)
impact_loss_gaussian_ws_kernel(const __grid_constant__ GaussParams p, const int S, const int W, const int lanes,
                               const int n_prefetch) {
    constexpr int NT = 128;
    constexpr int kRow = D * (int)sizeof(float);
    constexpr int kSlab = (int)ws_slab_pitch(NT, kRow);  // rows keep their place inside their 16-byte granule
    constexpr int kStageBytes = (int)gaussian_ws_stage_bytes<D>();
    constexpr float kLog2e = 1.4426950408889634f;
    constexpr float kHalfLog2Pi = 0.91893853320467274178f;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kWsMaxStages], empty_bar[kWsMaxStages];
    __shared__ unsigned int tickets_s, tag_s;
    __shared__ float2 warp_agg[C][NT / 32];
    __shared__ __align__(16) float red[C][NT / 32][8];
    __shared__ int abort_s;
    __shared__ float carry_s[C];

    const int tid = threadIdx.x, lane = tid & 31;
    const LossScalars& k = p.k;
    const TileGeometry& g = p.geo;
    const long long total_tiles = kLong ? g.nchunks * g.ntiles : g.nchunks;
    const int n_tiles = (int)((total_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x);
    const int rows_full = kLong ? NT : g.G * (int)g.T;
    const long long total_rows = g.B * g.T;
    const long long agg_stride = g.tile_major ? 2 * g.B : 2;  // slots between a tile's aggregate and that of the tile after it in time
    auto place_of = [&](int n) { return tile_place<kLong, NT>(g, n, rows_full, total_rows); };

    if (tid >= C * NT) {
        // ---- producer warp ----------------------------------------------------------------------------------
        const float* const src[5] = {p.learner_mean, p.learner_logstd, p.target_mean, p.target_logstd, p.actions};
        const int n_first = n_tiles < W ? n_tiles : W;
        const long long tensor_bytes = total_rows * kRow;
        // the block's first tiles are asked for in L2 before the stream dependency resolves, unless the launch's
        // companion kernel has done so already (see the categorical kernel): lane a takes array a
        if (n_prefetch > 0) {
            const void* base = nullptr;
            long long pitch = 4;
            if (lane < 5) { base = src[lane]; pitch = kRow; }
            else if (lane == 5) base = p.worker_logp;
            else if (lane == 6) base = p.rewards;
            else if (lane == 7) base = p.discounts;
            else if (lane == 8) base = p.values;
            const int n_pf = n_tiles < n_prefetch ? n_tiles : n_prefetch;
            for (int n = 0; n < n_pf; ++n) {
                const Place pc = place_of(n);
                if (base) dev::prefetch_range_l2(base, pc.row0 * pitch, (uint32_t)(pc.nrows * pitch), total_rows * pitch);
            }
        }
        if (lane < S) {
            dev::mbarrier_init_nofence(&full_bar[lane], 1);
            dev::mbarrier_init_nofence(&empty_bar[lane], NT / 32);
        }
        if (lane == 0) { abort_s = 0; tickets_s = 0u; }
        dev::fence_mbarrier_init();
        __syncwarp();

        // One slab of a tile into stage s (protocol, widened copies and in-order issue as in the categorical
        // kernel): lane l < 4 owns the round's l-th tile, requests its first slab, makes the barrier's arrival
        // with the bytes of all five slabs and fetches the bytes of a last, partial granule of the tensors; lanes
        // l + 4, l + 8, l + 12, l + 16 request the tile's other slabs.
        struct SlabRequest {
            unsigned char* d;      // the stage
            long long first;       // byte offset of the tile's first granule in each of the five tensors
            uint32_t span, tail;   // dev::WideRange
        };
        auto request_for = [&](const Place& pc, int s) {
            const dev::WideRange w = dev::widen_range(pc.row0 * (long long)kRow, (uint32_t)pc.nrows * kRow, tensor_bytes);
            SlabRequest r;
            r.d = smem_raw + s * kStageBytes;
            r.first = w.first;
            r.span = w.span;
            r.tail = w.tail;
            return r;
        };
        auto send_slab = [&](const SlabRequest& r, int s, int q) {
            uint64_t* const bar = &full_bar[s];
            const unsigned char* const gq = reinterpret_cast<const unsigned char*>(src[q]) + r.first;
            if (q == 0) {
                if (r.tail) {
#pragma unroll
                    for (int j = 0; j < 5; ++j) {
                        const unsigned char* const gj = reinterpret_cast<const unsigned char*>(src[j]) + r.first;
                        for (uint32_t i = 0; i < r.tail; ++i) r.d[j * kSlab + r.span + i] = gj[r.span + i];
                    }
                    dev::fence_async_shared();
                }
                if (r.span) dev::mbarrier_expect_tx(bar, 5 * r.span);
                else dev::mbarrier_arrive(bar);
            }
            if (r.span) dev::bulk_load(r.d + q * kSlab, gq, r.span, bar);
        };
        const int sub = lane & 3, q_lane = lane >> 2;
        const bool sends = q_lane < 5;
        const SlabRequest first = request_for(place_of(sub < n_first ? sub : 0), sub);

        grid_dependency_wait();

        // the first W tiles need no wait (tile n goes to stage n), four at a time
        if (sends && sub < n_first) send_slab(first, sub, q_lane);
        for (int base = 4; base < n_first; base += 4)
            if (sends && base + sub < n_first) send_slab(request_for(place_of(base + sub), base + sub), base + sub, q_lane);
        __syncthreads();  // the barriers are set up: the consumer warps may use them
        const unsigned int tag = dev::launch_tag(p.counter);  // (asked for now, needed after the last tile has left)
        for (int base = n_first; base < n_tiles; base += lanes) {
            const int n = base + sub;
            bool pending = sends && sub < lanes && n < n_tiles;
            const int cyc = n / S, s = n - cyc * S;
            const int wcyc = (n - W) / S, ws = (n - W) - wcyc * S;
            const SlabRequest req = request_for(place_of(pending ? n : 0), s);
            for (unsigned int spin = 0; spin < (1u << 22); ++spin) {
                const bool ready = q_lane == 0 && pending && (cyc == 0 || dev::mbarrier_test(&empty_bar[s], (uint32_t)(cyc - 1) & 1u)) &&
                                   dev::mbarrier_test(&full_bar[ws], (uint32_t)wcyc & 1u);
                const unsigned int waiting = __ballot_sync(0xffffffffu, q_lane == 0 && pending && !ready);
                bool go = ready && (waiting & ((1u << sub) - 1u)) == 0u;
                go = __shfl_sync(0xffffffffu, go, sub);  // the owner decides for all lanes of its tile
                if (go && pending) {
                    send_slab(req, s, q_lane);
                    pending = false;
                }
                if (!__any_sync(0xffffffffu, pending)) break;
                if (*reinterpret_cast<volatile int*>(&abort_s)) break;
                __nanosleep(32);
            }
            if (__any_sync(0xffffffffu, pending)) {  // a stage never came back, or a tile never landed
                if (lane == 0) {
                    atomicExch(p.counter + 1, 1u);
                    *reinterpret_cast<volatile int*>(&abort_s) = 1;
                }
                break;
            }
        }
        __syncwarp();
        // this launch's tag for whoever publishes the block's sums, and the warp's own ticket
        if (lane == 0) tag_s = tag;
        dev::draw_ticket_and_publish<C, NT / 32>(&tickets_s, &tag_s, red, p.tagged_rows);
        return;
    }

    // ---- consumer groups ------------------------------------------------------------------
    const int grp = tid >> 7, gtid = tid & (NT - 1), gwarp = gtid >> 5;
    const int bar_id = grp + 1;
    const bool want_kl = (k.kl_coef != 0.0f);

    int q = 0, ts = gtid;
    if (!kLong && g.G > 1) { q = gtid / (int)g.T; ts = gtid - q * (int)g.T; }
    struct Mine {
        long long row, traj;
        bool active, last_step;
        Place pc;
    };
    auto mine_in = [&](int n) {
        Mine m;
        m.pc = place_of(n < n_tiles ? n : 0);
        m.row = m.pc.row0 + gtid;
        m.traj = m.pc.traj + q;
        m.active = n < n_tiles && gtid < m.pc.nrows;
        m.last_step = kLong ? (m.pc.r == 0 && gtid == m.pc.nrows - 1) : (ts == (int)g.T - 1);
        return m;
    };

    struct StepRaw {
        float l_worker, reward, discount, value, value_next;
    };
    auto load_scalars = [&](const Mine& m) {
        StepRaw x;
        x.l_worker = 0.0f; x.reward = 0.0f; x.discount = 0.0f; x.value = 0.0f; x.value_next = 0.0f;
        if (m.active) {
            const long long r = m.row;
            x.l_worker = p.worker_logp[r];
            x.reward = p.rewards[r];
            x.discount = p.discounts[r];
            x.value = p.values[r];
            x.value_next = m.last_step ? p.bootstrap[m.traj] : p.values[r + 1];
        }
        return x;
    };

    float t_surr = 0.0f, t_val = 0.0f, t_ent = 0.0f, t_ratio = 0.0f, t_kl = 0.0f;
    int n_clip = 0, n_trunc = 0;
    auto hand_over_sums = [&]() {
        dev::hand_over_warp_sums<C, NT / 32>(t_surr, t_val, t_ent, t_ratio, t_kl, want_kl, n_clip, n_trunc, red[grp][gwarp],
                                             &tickets_s, &tag_s, red, p.tagged_rows);
    };
    bool pending = false;
    int pending_stage = 0;

    grid_dependency_wait();
    Mine me = mine_in(grp);
    StepRaw cur = load_scalars(me);
    __syncthreads();  // the producer warp has set up the barriers
    int s = grp % S;
    uint32_t ph = (uint32_t)(grp / S) & 1u;

    for (int n = grp; n < n_tiles; n += C) {
        const Mine me_next = mine_in(n + C);
        const StepRaw nxt = load_scalars(me_next);
        const bool active = me.active;
        const long long row = me.row;
        if (lane == 0 && pending) {
            dev::bulk_store_wait_read();
            dev::mbarrier_arrive(&empty_bar[pending_stage]);
            pending = false;
        }
        // (long trajectories) one early look at the aggregates of the later tiles of this tile's trajectory: with
        // many trajectories they were published a round ago, and reading them now keeps that trip to L2 off the
        // path between this tile's scan and its gradients
        // (only where tiles are numbered tile-major; the values are first looked at after the scan)
        const bool peeked = kLong && g.tile_major && gwarp == 0 && me.pc.r > lane;
        unsigned long long early_a = 0, early_b = 0;
        if (peeked)
            dev::load_aggregate(p.tile_aggregates + 2 * ((long long)blockIdx.x + (long long)n * gridDim.x), agg_stride,
                                me.pc.r - lane, early_a, early_b);
        if (!dev::mbarrier_wait(&full_bar[s], ph, &abort_s)) atomicExch(p.counter + 1, 1u);

        // the tile's first row starts (row0 * kRow) mod 16 bytes into each slab
        unsigned char* const stage = smem_raw + s * kStageBytes + ((uint32_t)(me.pc.row0 * kRow) & 15u);
        float* const r_mu = reinterpret_cast<float*>(stage) + gtid * D;              // learner mean -> dmean
        float* const r_ls = reinterpret_cast<float*>(stage + kSlab) + gtid * D;      // learner log-std -> dlogstd
        const float* const r_mt = reinterpret_cast<const float*>(stage + 2 * kSlab) + gtid * D;
        const float* const r_lt = reinterpret_cast<const float*>(stage + 3 * kSlab) + gtid * D;
        const float* const r_ac = reinterpret_cast<const float*>(stage + 4 * kSlab) + gtid * D;
        dev::StepIn st;
        st.reward = cur.reward;
        st.discount = cur.discount;
        st.value = cur.value;
        st.value_next = cur.value_next;
        st.last_step = me.last_step;

        // ---- row pass (every thread; rows beyond the tile hold stale bytes and are masked)
        float ent, kl = 0.0f;
        {
            // log-probabilities: D-term sums of magnitude tens that end up in exponents, so they are
            // accumulated in fp64
            double lth = 0.0, ltg = 0.0;
            float ls_sum = 0.0f;
#pragma unroll
            for (int j = 0; j < D; ++j) {
                const float ls = r_ls[j], lt = r_lt[j], ac = r_ac[j], mu = r_mu[j], mt = r_mt[j];
                const float inv_s = dev::exp2_fast(-ls * kLog2e), inv_st = dev::exp2_fast(-lt * kLog2e);
                const float z1 = (ac - mu) * inv_s;
                const float z2 = (ac - mt) * inv_st;
                lth += (double)fmaf(-0.5f * z1, z1, -ls);
                ltg += (double)fmaf(-0.5f * z2, z2, -lt);
                ls_sum += ls;
                if (want_kl) {  // KL(target || learner), per dimension
                    const float dm = (mt - mu) * inv_s;
                    const float sr = dev::exp2_fast((lt - ls) * kLog2e);
                    kl += (ls - lt) + 0.5f * fmaf(sr, sr, dm * dm) - 0.5f;
                }
            }
            ent = ls_sum + (float)D * (kHalfLog2Pi + 0.5f);
            const double shift = (double)cur.l_worker + (double)D * (double)kHalfLog2Pi;
            // everything downstream works on log-probabilities relative to the worker's
            st.l_theta = (float)(lth - shift);
            st.l_target = (float)(ltg - shift);
            st.l_worker = 0.0f;
            st.l_shift = cur.l_worker;
        }
        float fa, fb;
        const bool truncated = dev::recursion_map(st, k, fa, fb);
        if (!active) { fa = 1.0f; fb = 0.0f; }
        float adv;
        if (!kLong) {
            adv = dev::suffix_affine_scan_group<NT>(fa, fb, warp_agg[grp], st.adv_next, bar_id);
        } else {
            float ma, mb, la, lb;
            dev::suffix_affine_maps_group<NT>(fa, fb, warp_agg[grp], ma, mb, la, lb, bar_id);
            const long long gtile = (long long)blockIdx.x + (long long)n * gridDim.x;
            if (gtid == 0) dev::publish_tile_aggregate(p.tile_aggregates + 2 * gtile, ma, mb, dev::launch_tag(p.counter));
            float carry = 0.0f;
            if (me.pc.r > 0) {  // uniform over the group
                if (gwarp == 0) {
                    const float c = dev::compose_later_aggregates(p.tile_aggregates + 2 * gtile, agg_stride, me.pc.r,
                                                                  dev::launch_tag(p.counter), &abort_s, peeked,
                                                                  early_a, early_b);
                    if (lane == 0) carry_s[grp] = c;
                }
                asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
                carry = carry_s[grp];
            }
            adv = fmaf(ma, carry, mb);
            const float below = __shfl_down_sync(0xffffffffu, adv, 1);
            st.adv_next = (lane == 31) ? fmaf(la, carry, lb) : below;
        }

        float surr, ratio;
        bool clipped;
        const float wpg = dev::surrogate(st, k, adv, surr, ratio, clipped);
        if (active) {
            t_surr += surr;
            t_val = fmaf(0.5f * adv, adv, t_val);
            t_ent += ent;
            t_ratio += ratio;
            t_kl += kl;
        }
        n_clip += __popc(__ballot_sync(0xffffffffu, active && clipped));
        n_trunc += __popc(__ballot_sync(0xffffffffu, active && truncated));
        if (n + C >= n_tiles) hand_over_sums();

        // ---- gradients, in place over the learner's slabs
        {
            const float w1 = wpg * k.inv_M, ce = k.ent_coef * k.inv_M, ck = k.kl_coef * k.inv_M;
#pragma unroll
            for (int j = 0; j < D; ++j) {
                const float ls = r_ls[j], mu = r_mu[j];
                const float inv_s = dev::exp2_fast(-ls * kLog2e);
                const float z = (r_ac[j] - mu) * inv_s;  // (a - mu) / sigma
                // d log pi / d mu = z / sigma ;  d log pi / d logstd = z^2 - 1 ;  d H / d logstd = 1
                float gm = -w1 * z;
                float gs = -w1 * fmaf(z, z, -1.0f) - ce;
                if (want_kl) {
                    const float dm = (mu - r_mt[j]) * inv_s;
                    const float sr = dev::exp2_fast((r_lt[j] - ls) * kLog2e);
                    gm = fmaf(ck, dm, gm);
                    gs = fmaf(ck, 1.0f - fmaf(sr, sr, dm * dm), gs);
                }
                r_mu[j] = gm * inv_s;
                r_ls[j] = gs;
            }
            if (active) {
                p.dvalues[row] = -k.vf_coef * k.inv_M * adv;
                if (p.vtarget) p.vtarget[row] = st.value + adv;
                if (p.advantage) p.advantage[row] = adv;
            }
        }
        // ---- each warp sends its own 32 rows of both gradient slabs
        {
            const long long wrow0 = row - lane;
            const int left = me.pc.nrows - (gtid - lane);
            const int wrows = left > 32 ? 32 : (left > 0 ? left : 0);
            unsigned char* const gm = reinterpret_cast<unsigned char*>(p.dmean) + wrow0 * (long long)kRow;
            unsigned char* const gs = reinterpret_cast<unsigned char*>(p.dlogstd) + wrow0 * (long long)kRow;
            const unsigned char* const src_m = stage + (gtid - lane) * kRow;
            bool stored = dev::warp_send_bytes(gm, src_m, (uint32_t)wrows * kRow, true);
            if (dev::warp_send_bytes(gs, src_m + kSlab, (uint32_t)wrows * kRow, false)) stored = true;  // (fenced above)
            if (lane == 0) {
                if (stored) {
                    pending = n_tiles > S;  // a block with no more tiles than stages never needs a stage back
                    pending_stage = s;
                } else {
                    dev::mbarrier_arrive(&empty_bar[s]);
                }
            }
        }
        cur = nxt;
        me = me_next;
        s += C;
        while (s >= S) { s -= S; ph ^= 1u; }
    }

    if (grp >= n_tiles) hand_over_sums();
    if (blockIdx.x == 0 && grp == n_tiles % C) {
        if (!dev::reduce_tagged_rows<NT>(p.tagged_rows, (int)gridDim.x, dev::launch_tag(p.counter), p.counter,
                                         p.loss_terms, k.vf_coef, k.ent_coef, k.kl_coef, k.steps_total,
                                         gtid, bar_id, &abort_s))
            if (gtid == 0) atomicExch(p.counter + 1, 1u);
    }
    if (lane == 0) dev::bulk_store_wait_read();
}

// ------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------
constexpr int kMaxGridBlocks = 4096;  // upper bound on blocks of a loss launch (sizes the workspace)
constexpr size_t kCounterBytes = 256; // words after the partials: [0] completion counter, [1] error flag, [2] launch number
// Long trajectories (T > 128 steps): two (value, tag) pairs per 128-step tile, after everything else.
constexpr int kMinTileRows = 64;  // the smallest tile of a persistent kernel
size_t tile_aggregate_bytes(int64_t B, int64_t T) {
    if (T <= kMinTileRows) return 0;
    return (size_t)B * (size_t)((T + kMinTileRows - 1) / kMinTileRows) * 2 * sizeof(unsigned long long);
}
constexpr int kMaxTaggedRows = 1024;  // rows of eight (value, tag) pairs after the counter words: one per block of the persistent kernel

constexpr size_t kWorkspaceFixedBytes = (size_t)kMaxGridBlocks * 8 * sizeof(float) + kCounterBytes +
                                        (size_t)kMaxTaggedRows * 8 * sizeof(unsigned long long);

int pad_odd(int w) { return (w & 1) ? w : w + 1; }

// Shared memory of the runtime-width categorical kernel: two input slabs, and a gradient slab
// of its own when gradients and logits differ in element size.
size_t generic_categorical_smem(int nt, int A, size_t in_elem, size_t out_elem) {
    return (size_t)nt * A * (2 * in_elem + (in_elem == out_elem ? 0 : out_elem));
}
int pick_nt_categorical(int A, size_t in_elem, size_t out_elem, size_t budget) {
    for (int nt : {128, 64})
        if (generic_categorical_smem(nt, A, in_elem, out_elem) <= budget) return nt;
    return 32;
}

// Threads per block = rows per tile: as many as keep a tile's staged slabs within
// `budget` bytes of shared memory, so that several blocks stay resident per SM.
int pick_nt(int width_padded, int n_slabs, size_t budget) {
    for (int nt : {128, 64}) {
        if ((size_t)nt * width_padded * n_slabs * sizeof(float) <= budget) return nt;
    }
    return 32;
}

TileGeometry make_geometry(int64_t B, int64_t T, int nt) {
    TileGeometry g;
    g.tile_major = 0;
    g.B = B;
    g.T = T;
    if (T <= nt) {
        g.G = (int)(nt / T);
        g.ntiles = 1;
        g.nchunks = (B + g.G - 1) / g.G;
    } else {
        g.G = 1;
        g.ntiles = (int)((T + nt - 1) / nt);
        g.nchunks = B;
    }
    return g;
}

bool bad_scalar(float x) { return !(x >= 0.0f); }  // negative or NaN

int32_t fill_scalars(LossScalars& k, float rho_bar, float c_bar, float clip_eps,
                     const impact_coefficients* coef, int64_t B, int64_t T) {
    if (bad_scalar(rho_bar) || bad_scalar(c_bar) || bad_scalar(clip_eps)) return IMPACT_ERR_INVALID_ARG;
    if (!(coef->rho_tw > 0.0f) || !isfinite(coef->vf_coef) || !isfinite(coef->ent_coef) ||
        !isfinite(coef->kl_coef) || !isfinite(coef->lambda_))
        return IMPACT_ERR_INVALID_ARG;
    if (coef->is_source < IMPACT_IS_TARGET_OVER_WORKER || coef->is_source > IMPACT_IS_NONE) return IMPACT_ERR_INVALID_ARG;
    if (coef->objective != IMPACT_OBJECTIVE_CLIPPED_SURROGATE && coef->objective != IMPACT_OBJECTIVE_VTRACE_PG)
        return IMPACT_ERR_INVALID_ARG;
    if (coef->ratio_mode < IMPACT_RATIO_R3 || coef->ratio_mode > IMPACT_RATIO_R2) return IMPACT_ERR_INVALID_ARG;
    k.rho_bar = rho_bar;
    k.c_bar = c_bar;
    k.clip_lo = 1.0f - clip_eps;
    k.clip_hi = 1.0f + clip_eps;
    k.vf_coef = coef->vf_coef;
    k.ent_coef = coef->ent_coef;
    k.kl_coef = coef->kl_coef;
    k.lambda_ = coef->lambda_;
    k.log_rho_tw = (float)log((double)coef->rho_tw);
    const double own = (double)B * (double)T;
    if (coef->global_steps != 0 && (double)coef->global_steps < own) return IMPACT_ERR_INVALID_ARG;
    k.steps_total = coef->global_steps != 0 ? (double)coef->global_steps : own;
    k.inv_M = (float)(1.0 / k.steps_total);
    k.is_source = coef->is_source;
    k.ratio_mode = coef->ratio_mode;
    k.objective = coef->objective;
    return IMPACT_OK;
}

// Blocks to launch: every chunk gets its own block while all of them can be resident at
// once; beyond that, a resident-sized grid walks the chunks.
template <typename Kernel>
int32_t grid_for(Kernel kernel, int nt, size_t smem, long long nchunks, const DeviceInfo* di, int* grid) {
    struct Key { const void* fn; size_t smem; int dev; int per_sm; };
    static thread_local Key cache[16];
    static thread_local int ncache = 0;
    int per_sm = -1;
    for (int i = 0; i < ncache; ++i)
        if (cache[i].fn == (const void*)kernel && cache[i].smem == smem && cache[i].dev == di->device)
            per_sm = cache[i].per_sm;
    if (per_sm < 0) {
        if (smem > 48 * 1024)
            IMPACT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        IMPACT_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, nt, smem));
        if (per_sm < 1) return IMPACT_ERR_UNSUPPORTED;
        if (ncache < 16) cache[ncache++] = Key{(const void*)kernel, smem, di->device, per_sm};
    }
    long long resident = (long long)per_sm * di->sm_count;
    if (resident > kMaxGridBlocks) resident = kMaxGridBlocks;
    *grid = (int)(nchunks < resident ? nchunks : resident);
    return IMPACT_OK;
}

template <typename LT, typename GT, int NT>
int32_t launch_categorical(const CatParams& p, const DeviceInfo* di, cudaStream_t stream) {
    auto kernel = impact_loss_categorical_kernel<LT, GT, NT>;
    const size_t smem = generic_categorical_smem(NT, p.A, sizeof(LT), sizeof(GT));
    int grid = 0;
    int32_t st = grid_for(kernel, NT, smem, p.geo.nchunks, di, &grid);
    if (st != IMPACT_OK) return st;
    IMPACT_CUDA_TRY(launch_serialized(kernel, dim3(grid), dim3(NT), smem, stream, p));
    return IMPACT_OK;
}

template <typename LT, typename GT>
int32_t dispatch_nt(const CatParams& p, int nt, const DeviceInfo* di, cudaStream_t stream) {
    switch (nt) {
        case 128: return launch_categorical<LT, GT, 128>(p, di, stream);
        case 64: return launch_categorical<LT, GT, 64>(p, di, stream);
        default: return launch_categorical<LT, GT, 32>(p, di, stream);
    }
}

// The copy of the target logits for the kernels that do not write it themselves: an ordinary device copy ahead
// of the launch.
int32_t copy_target_logits(const CatParams& p, size_t elem, cudaStream_t stream) {
    if (!p.target_copy) return IMPACT_OK;
    const size_t bytes = (size_t)p.geo.B * (size_t)p.geo.T * (size_t)p.A * elem;
    IMPACT_CUDA_TRY(cudaMemcpyAsync(p.target_copy, p.target_logits, bytes, cudaMemcpyDeviceToDevice, stream));
    return IMPACT_OK;
}

// Tiles the producer keeps in flight and stages of the ring, for tiles of `tile_in_bytes` bytes of logits.
// Bytes in flight per SM (IMPACT_OPT_WINDOW_BYTES; 0 = chosen here): 72 KB where a block streams many tiles (over
// 148 SMs that covers HBM's latency at full bandwidth; measured: 64 KB and more reach the copy rate, 48 KB stop at
// 0.9 of it), 48 KB where a block has only a few (a bigger first burst makes every tile of it land later, and the
// first tile's landing is what such a launch waits for).  Beyond the window there is room for the tiles being
// worked on and being stored.  The barrier protocol needs stages >= in_flight + groups, or exactly one stage per
// group (then the stage's previous tile is the one the same group worked on last); 0 stages = no valid shape.
void ws_ring_shape(size_t stage_bytes, size_t tile_in_bytes, int groups, int max_smem, long long tiles_per_block,
                   int* stages, int* in_flight) {
    size_t window = (size_t)option(IMPACT_OPT_WINDOW_BYTES);
    if (window == 0) window = tiles_per_block <= 8 ? 48 * 1024 : 72 * 1024;
    int w = (int)((window + tile_in_bytes - 1) / tile_in_bytes);
    if (w < 2) w = 2;
    if (w > 8) w = 8;
    int s = w + groups + 3;
    if (s > kWsMaxStages) s = kWsMaxStages;
    const int fit = (int)((size_t)(max_smem - 4096) / stage_bytes);  // 4 KB left for static shared memory
    if (s > fit) s = fit;
    if (tiles_per_block <= s) {
        // no stage is used twice: every barrier sees one phase only, and any number of tiles may be in flight
        if (w > s) w = s;
    } else if (s > groups) {
        if (w > s - groups) w = s - groups;
    } else if (s == groups) {
        if (w > s) w = s;
    } else {
        s = 0;
    }
    *stages = s;
    *in_flight = w;
}

// How a persistent kernel is launched for a batch of `tiles` tiles on `grid` blocks.
struct WsPlan {
    int prefetch_tiles;  // tiles per block asked for in L2 ahead of time
    bool companion;      // by a companion kernel enqueued before the loss kernel (else by the loss kernel's first warp)
};
WsPlan ws_plan(long long tiles, long long grid, size_t tile_bytes, int in_flight, bool allow_companion) {
    WsPlan pl;
    const long long per_block = (tiles + grid - 1) / grid;
    const long long budget = option(IMPACT_OPT_PREFETCH_BYTES);
    long long pf = budget / (grid * (long long)tile_bytes);
    // Asking L2 for tiles ahead of time goes through the copy engine like the tiles themselves, so it pays only
    // where requests are large (measured: with 12-21 KB tiles a short launch gains half a microsecond from its
    // companion and a third from asking itself; with 3-9 KB tiles either costs 5-15 %).  The companion pays where a
    // launch is short: a block has a handful of tiles, all within the budget.  A long launch is bound by HBM either
    // way, and asking for many tiles far ahead of their use only competes with the tiles that are needed now.
    // Without a companion the loss kernel's first warp asks for the tiles it is about to request anyway (more than
    // that sits in the copy engine's queue ahead of the requests themselves).
    const bool large_tiles = tile_bytes >= 10 * 1024;
    // (measured on 18 actions: a gain from five tiles per block on -- 8.3 -> 7.6 us at seven --, nothing at three
    // to four, a loss of a quarter of a microsecond at two)
    pl.companion = allow_companion && large_tiles && option(IMPACT_OPT_EARLY_PREFETCH) != 0 && pf >= per_block &&
                   per_block >= 4 && per_block <= 8;
    if (!large_tiles) pf = 0;
    if (!pl.companion && pf > in_flight) pf = in_flight;
    if (pf > per_block) pf = per_block;
    pl.prefetch_tiles = (int)pf;
    return pl;
}

int32_t launch_companion(const PrefetchList& pf, long long grid, cudaStream_t stream) {
    IMPACT_CUDA_TRY(launch_serialized(impact_prefetch_kernel, dim3((unsigned)grid), dim3(32), 0, stream, pf));
    return IMPACT_OK;
}

template <typename LT, typename GT, int A, bool kPlain, bool kLong>
int32_t launch_categorical_ws(const CatParams& p, const DeviceInfo* di, cudaStream_t stream) {
    // Consumer groups: four with every switch compiled in (96 registers); five in the default configuration (80
    // registers, no spills); six there for small action sets, which are bound by arithmetic, not bytes, and fit 72.
    // Wide rows (A = 64): tiles of 64 steps, six groups of 64 threads.
    constexpr int NT = ws_tile_rows(A);
    // One step of a tile per thread.  (Two -- groups of 64 threads, seven groups, 128 registers -- execute 18 %
    // fewer instructions on 18 actions and 27 % fewer on 6, everything paid per thread and tile being paid half as
    // often, but a launch takes 0.3 us longer on 131 072 steps and 7 % longer on a million, and small action sets
    // lose 7-20 % with eight to twelve such groups: a tile's rows then wait on half as many warps, and what
    // bounds a launch is how long a tile takes, not how many instructions the SM issues.)
    constexpr int R = 1;
    constexpr int C = A > 32 ? 6 : (!kPlain ? kWsGroups : (A <= 9 ? kWsGroups + 2 : kWsGroups + 1));
    // (inputs named by a device record: compiled for trajectories that fit a tile only)
    if (p.indirect && kLong) return IMPACT_ERR_UNSUPPORTED;
    auto kernel = impact_loss_categorical_ws_kernel<LT, GT, A, C, kPlain, kLong, NT, false, R>;
    if constexpr (!kLong)
        if (p.indirect) kernel = impact_loss_categorical_ws_kernel<LT, GT, A, C, kPlain, kLong, NT, true, R>;
    const size_t stage = ws_stage_bytes<LT, GT, A, NT>();
    const long long tiles = kLong ? p.geo.nchunks * p.geo.ntiles : p.geo.nchunks;
    long long grid = tiles < di->sm_count ? tiles : di->sm_count;
    if (grid > kMaxTaggedRows) grid = kMaxTaggedRows;  // one tagged row per block
    int S = 0, W = 0;
    ws_ring_shape(stage, 2 * (size_t)NT * A * sizeof(LT), C, di->max_smem_optin, (tiles + grid - 1) / grid, &S, &W);
    if (S < 1 || W < 1) return IMPACT_ERR_UNSUPPORTED;

    const size_t smem = (size_t)S * stage;
    static thread_local int configured_device[2] = {-1, -1};
    int& configured = configured_device[p.indirect ? 1 : 0];
    if (configured != di->device) {  // once per device: room for the largest ring any window setting asks for
        IMPACT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, di->max_smem_optin - 4096));
        configured = di->device;
    }
    const int lanes = (S - W) < 4 ? ((S - W) < 1 ? 1 : (S - W)) : 4;  // producer lanes that request tiles side by side
    CatParams q = p;
    // tile-major once every block has a trajectory of its own: the aggregates a tile needs are then a round old
    q.geo.tile_major = (kLong && p.geo.B >= grid) ? 1 : 0;
    const int rows_full = kLong ? NT : q.geo.G * (int)q.geo.T;
    // (rows wider than 32 actions: the companion gains nothing with fp32 logits and doubles a launch with bf16 ones
    // -- 27 against 14 us at 65 536 steps --, so such launches ask for their first tiles themselves)
    WsPlan plan_ = ws_plan(tiles, grid, (size_t)rows_full * (2 * A * sizeof(LT) + 20), W, A <= 32);
    if (p.indirect) { plan_.companion = false; plan_.prefetch_tiles = 0; }  // (addresses unknown on the host)
    const WsPlan plan = plan_;
    if (plan.companion) {
        PrefetchList pf = {};
        const void* bases[7] = {p.learner_logits, p.target_logits, p.actions, p.worker_logp, p.rewards, p.discounts, p.values};
        for (int i = 0; i < 7; ++i) {
            pf.base[i] = bases[i];
            pf.row_bytes[i] = i < 2 ? A * (int)sizeof(LT) : 4;
        }
        pf.n_arrays = 7;
        pf.n_tiles_max = plan.prefetch_tiles;
        pf.nt = NT;
        pf.is_long = kLong ? 1 : 0;
        pf.geo = q.geo;
        const int32_t st = launch_companion(pf, grid, stream);
        if (st != IMPACT_OK) return st;
    }
    IMPACT_CUDA_TRY(launch_serialized(kernel, dim3((unsigned)grid), dim3(C * (NT / R) + 32), smem, stream, q, S, W, lanes,
                                      plan.companion ? 0 : plan.prefetch_tiles));
    return IMPACT_OK;
}

// The persistent kernel serves every batch: trajectories that fit a tile (T <= 128) and, where the caller's
// scratch has room for the tiles' aggregates, longer ones; the kernel that sweeps a long trajectory tile by
// tile inside one block remains for scratch without that room.
template <typename LT, typename GT, int A>
int32_t launch_categorical_reg(const CatParams& p, const DeviceInfo* di, cudaStream_t stream) {
    if (p.geo.ntiles == 1) {
        const bool plain = p.k.kl_coef == 0.0f && p.k.objective == IMPACT_OBJECTIVE_CLIPPED_SURROGATE &&
                           p.k.is_source == IMPACT_IS_TARGET_OVER_WORKER && p.k.ratio_mode == IMPACT_RATIO_R3 &&
                           !p.vtarget && !p.advantage;
        if (plain) return launch_categorical_ws<LT, GT, A, true, false>(p, di, stream);
        return launch_categorical_ws<LT, GT, A, false, false>(p, di, stream);
    }
    // Split across blocks while there are too few trajectories to give every consumer group of the device one of
    // its own; from there on the sweep inside a block keeps the device busy without any exchange between tiles.
    if constexpr (A > 32) {  // no sweeping kernel for wide rows: run_categorical sends long trajectories here only with aggregates
        return launch_categorical_ws<LT, GT, A, false, true>(p, di, stream);
    } else {
        // with trajectories for every consumer group of the device the sweep inside a block is a little faster still
        if (p.tile_aggregates && p.geo.B < (long long)kWsGroups * di->sm_count)
            return launch_categorical_ws<LT, GT, A, false, true>(p, di, stream);
        if (p.indirect) return IMPACT_ERR_UNSUPPORTED;  // the sweeping kernel takes its pointers from the call only
        auto kernel = impact_loss_categorical_reg_kernel<LT, GT, A>;
        const size_t smem = reg_kernel_smem<LT, GT, A>();
        int grid = 0;
        int32_t st = grid_for(kernel, kRegTileRows, smem, p.geo.nchunks, di, &grid);
        if (st != IMPACT_OK) return st;
        st = copy_target_logits(p, sizeof(LT), stream);  // this kernel does not write the copy itself
        if (st != IMPACT_OK) return st;
        IMPACT_CUDA_TRY(launch_serialized(kernel, dim3(grid), dim3(kRegTileRows), smem, stream, p));
        return IMPACT_OK;
    }
}

// Action counts with a compiled kernel (the Atari action sets, and 64).
constexpr bool has_reg_kernel(int A) { return A == 4 || A == 6 || A == 9 || A == 18 || A == 64; }

template <typename LT, typename GT>
int32_t dispatch_reg(const CatParams& p, const DeviceInfo* di, cudaStream_t stream) {
    switch (p.A) {
        case 4: return launch_categorical_reg<LT, GT, 4>(p, di, stream);
        case 6: return launch_categorical_reg<LT, GT, 6>(p, di, stream);
        case 9: return launch_categorical_reg<LT, GT, 9>(p, di, stream);
        case 64: return launch_categorical_reg<LT, GT, 64>(p, di, stream);
        default: return launch_categorical_reg<LT, GT, 18>(p, di, stream);
    }
}

// Steps per tile of the kernel that run_categorical picks for this call.
int categorical_tile_rows(int A, bool logits_bf16, bool grads_bf16, bool long_without_aggregates) {
    if (has_reg_kernel(A) && !(A > 32 && long_without_aggregates)) return ws_tile_rows(A);
    return pick_nt_categorical(A, logits_bf16 ? 2 : 4, grads_bf16 ? 2 : 4, 72 * 1024);
}

// Picks the kernel for a categorical call: the register-resident one where it exists, else
// the generic one.  `p` arrives complete except for As and geo.
int32_t run_categorical(CatParams& p, int64_t B, int64_t T, bool logits_bf16, bool grads_bf16,
                        const DeviceInfo* di, cudaStream_t s) {
    // (wide rows have no kernel that sweeps a long trajectory inside one block: without room for the tiles'
    // aggregates such a call takes the runtime-width kernel)
    const bool long_without_aggregates = T > ws_tile_rows(p.A) && !p.tile_aggregates;
    if (has_reg_kernel(p.A) && !(p.A > 32 && long_without_aggregates)) {
        p.As = p.A;
        p.geo = make_geometry(B, T, ws_tile_rows(p.A));
        if (!logits_bf16 && !grads_bf16) return dispatch_reg<float, float>(p, di, s);
        if (!logits_bf16 && grads_bf16) return dispatch_reg<float, __nv_bfloat16>(p, di, s);
        if (logits_bf16 && !grads_bf16) return dispatch_reg<__nv_bfloat16, float>(p, di, s);
        return dispatch_reg<__nv_bfloat16, __nv_bfloat16>(p, di, s);
    }
    if (p.indirect) return IMPACT_ERR_UNSUPPORTED;  // inputs named by a device record: the persistent kernel only
    p.As = p.A;
    const int nt = categorical_tile_rows(p.A, logits_bf16, grads_bf16, long_without_aggregates);
    p.geo = make_geometry(B, T, nt);
    {
        const int32_t st = copy_target_logits(p, logits_bf16 ? 2 : 4, s);  // the runtime-width kernel does not write it
        if (st != IMPACT_OK) return st;
    }
    if (!logits_bf16 && !grads_bf16) return dispatch_nt<float, float>(p, nt, di, s);
    if (!logits_bf16 && grads_bf16) return dispatch_nt<float, __nv_bfloat16>(p, nt, di, s);
    if (logits_bf16 && !grads_bf16) return dispatch_nt<__nv_bfloat16, float>(p, nt, di, s);
    return dispatch_nt<__nv_bfloat16, __nv_bfloat16>(p, nt, di, s);
}

template <int NT>
int32_t launch_gaussian(const GaussParams& p, const DeviceInfo* di, cudaStream_t stream) {
    auto kernel = impact_loss_gaussian_kernel<NT>;
    const size_t smem = (size_t)5 * NT * p.Ds * sizeof(float);
    int grid = 0;
    int32_t st = grid_for(kernel, NT, smem, p.geo.nchunks, di, &grid);
    if (st != IMPACT_OK) return st;
    IMPACT_CUDA_TRY(launch_serialized(kernel, dim3(grid), dim3(NT), smem, stream, p));
    return IMPACT_OK;
}

constexpr int kWsGroupsGaussian = 3;  // consumer groups: five slabs per tile leave room for five stages at D = 17

template <int D, bool kLong>
int32_t launch_gaussian_ws(const GaussParams& p, const DeviceInfo* di, cudaStream_t stream) {
    constexpr int C = kWsGroupsGaussian;
    auto kernel = impact_loss_gaussian_ws_kernel<D, C, kLong>;
    const size_t stage = gaussian_ws_stage_bytes<D>();
    const long long tiles = kLong ? p.geo.nchunks * p.geo.ntiles : p.geo.nchunks;
    long long grid = tiles < di->sm_count ? tiles : di->sm_count;
    if (grid > kMaxTaggedRows) grid = kMaxTaggedRows;  // one tagged row per block
    int S = 0, W = 0;
    ws_ring_shape(stage, stage, C, di->max_smem_optin, (tiles + grid - 1) / grid, &S, &W);
    if (S < 1 || W < 1) return IMPACT_ERR_UNSUPPORTED;
    const size_t smem = (size_t)S * stage;
    static thread_local int configured_device = -1;
    if (configured_device != di->device) {
        IMPACT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, di->max_smem_optin - 4096));
        configured_device = di->device;
    }
    const int lanes = (S - W) < 4 ? ((S - W) < 1 ? 1 : (S - W)) : 4;  // tiles the producer requests side by side
    GaussParams q = p;
    q.geo.tile_major = (kLong && p.geo.B >= grid) ? 1 : 0;
    const int rows_full = kLong ? 128 : q.geo.G * (int)q.geo.T;
    // (no companion here: measured on B = 512, T = 128, D = 17 it costs more of the copy engine's time than the
    // earlier start gains: 10.7 us per launch with it, 8.8 us without)
    const WsPlan plan = ws_plan(tiles, grid, (size_t)rows_full * (5 * D * sizeof(float) + 16), W, false);
    if (plan.companion) {
        PrefetchList pf = {};
        const void* bases[9] = {p.learner_mean, p.learner_logstd, p.target_mean, p.target_logstd, p.actions,
                                p.worker_logp, p.rewards, p.discounts, p.values};
        for (int i = 0; i < 9; ++i) {
            pf.base[i] = bases[i];
            pf.row_bytes[i] = i < 5 ? D * (int)sizeof(float) : 4;
        }
        pf.n_arrays = 9;
        pf.n_tiles_max = plan.prefetch_tiles;
        pf.nt = 128;
        pf.is_long = kLong ? 1 : 0;
        pf.geo = q.geo;
        const int32_t st = launch_companion(pf, grid, stream);
        if (st != IMPACT_OK) return st;
    }
    IMPACT_CUDA_TRY(launch_serialized(kernel, dim3((unsigned)grid), dim3(C * 128 + 32), smem, stream, q, S, W, lanes,
                                      plan.companion ? 0 : plan.prefetch_tiles));
    return IMPACT_OK;
}

template <int D>
int32_t launch_gaussian_reg(const GaussParams& p, const DeviceInfo* di, cudaStream_t stream) {
    if (p.geo.ntiles == 1) return launch_gaussian_ws<D, false>(p, di, stream);
    if (p.tile_aggregates) return launch_gaussian_ws<D, true>(p, di, stream);
    auto kernel = impact_loss_gaussian_reg_kernel<D>;
    const size_t smem = (size_t)5 * kRegTileRows * D * sizeof(float);
    int grid = 0;
    int32_t st = grid_for(kernel, kRegTileRows, smem, p.geo.nchunks, di, &grid);
    if (st != IMPACT_OK) return st;
    IMPACT_CUDA_TRY(launch_serialized(kernel, dim3(grid), dim3(kRegTileRows), smem, stream, p));
    return IMPACT_OK;
}

// Action dimensions with a compiled register-resident kernel (the MuJoCo tasks of Section 4.3).
constexpr bool has_gaussian_reg_kernel(int D) { return D == 3 || D == 6 || D == 17; }

}  // namespace
}  // namespace impact

using namespace impact;

extern "C" size_t impact_loss_workspace_bytes(int64_t B, int64_t T) {
    if (B <= 0 || T <= 0) return 0;
    return kWorkspaceFixedBytes + tile_aggregate_bytes(B, T);
}

extern "C" int32_t impact_loss_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    if (!workspace || !aligned16(workspace) || workspace_bytes == 0) return IMPACT_ERR_INVALID_ARG;
    IMPACT_CUDA_TRY(cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream)));
    return IMPACT_OK;
}

extern "C" int32_t impact_loss_workspace_status(const void* workspace, size_t workspace_bytes, int32_t* flag_out,
                                                void* stream) {
    if (!workspace || !flag_out || !aligned16(workspace)) return IMPACT_ERR_INVALID_ARG;
    if (workspace_bytes < impact_loss_workspace_bytes(1, 1)) return IMPACT_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const char* word = static_cast<const char*>(workspace) + (size_t)kMaxGridBlocks * 8 * sizeof(float) + sizeof(unsigned int);
    unsigned int flag = 0;
    IMPACT_CUDA_TRY(cudaMemcpyAsync(&flag, word, sizeof(flag), cudaMemcpyDeviceToHost, s));
    IMPACT_CUDA_TRY(cudaStreamSynchronize(s));
    *flag_out = (int32_t)flag;
    return IMPACT_OK;
}

static int32_t loss_fwd_bwd_impl(
    const void* learner_logits, const void* target_logits, const float* worker_logp,
    const int32_t* actions, const float* rewards, const float* discounts, const float* values,
    const float* bootstrap_values, float rho_bar, float c_bar, float clip_eps,
    const impact_coefficients* coef, int64_t B, int64_t T, int32_t A, int32_t logits_dtype,
    float* loss_terms, void* dlogits, float* dvalues, float* vtarget, float* advantage,
    void* workspace, size_t workspace_bytes, void* target_logits_copy, const impact_loss_inputs* indirect, void* stream) {
    if (!coef || !loss_terms || !dlogits || !dvalues || !workspace) return IMPACT_ERR_INVALID_ARG;
    if (indirect) {  // the inputs come from a record in device memory: the pointers passed here are not looked at
        if (!aligned16(indirect)) return IMPACT_ERR_INVALID_ARG;
        learner_logits = target_logits = nullptr;
        worker_logp = rewards = discounts = values = bootstrap_values = nullptr;
        actions = nullptr;
        target_logits_copy = nullptr;
    } else if (!learner_logits || !target_logits || !worker_logp || !actions || !rewards || !discounts || !values ||
               !bootstrap_values) {
        return IMPACT_ERR_INVALID_ARG;
    }
    if (B <= 0 || T <= 0 || A <= 0) return IMPACT_ERR_INVALID_ARG;
    const void* ptrs[] = {learner_logits, target_logits, worker_logp, actions, rewards, discounts,
                          values, bootstrap_values, loss_terms, dlogits, dvalues, workspace};
    for (const void* q : ptrs)
        if (!aligned16(q)) return IMPACT_ERR_INVALID_ARG;
    if ((vtarget && !aligned16(vtarget)) || (advantage && !aligned16(advantage))) return IMPACT_ERR_INVALID_ARG;
    if (target_logits_copy && (!aligned16(target_logits_copy) || target_logits_copy == target_logits))
        return IMPACT_ERR_INVALID_ARG;
    if (logits_dtype != IMPACT_DTYPE_F32 && logits_dtype != IMPACT_DTYPE_BF16) return IMPACT_ERR_INVALID_ARG;
    if (coef->dlogits_dtype != IMPACT_DTYPE_F32 && coef->dlogits_dtype != IMPACT_DTYPE_BF16)
        return IMPACT_ERR_INVALID_ARG;
    if (A > 512) return IMPACT_ERR_UNSUPPORTED;
    if ((double)B * (double)T * (double)A >= 1099511627776.0 || (double)B * (double)T >= 4.0e12)
        return IMPACT_ERR_UNSUPPORTED;
    if (workspace_bytes < kWorkspaceFixedBytes) return IMPACT_ERR_WORKSPACE_TOO_SMALL;

    CatParams p = {};
    int32_t st = fill_scalars(p.k, rho_bar, c_bar, clip_eps, coef, B, T);
    if (st != IMPACT_OK) return st;
    const DeviceInfo* di = current_device_info();
    if (!di) return IMPACT_ERR_CUDA;

    p.learner_logits = learner_logits;
    p.target_logits = target_logits;
    p.worker_logp = worker_logp;
    p.actions = actions;
    p.rewards = rewards;
    p.discounts = discounts;
    p.values = values;
    p.bootstrap = bootstrap_values;
    p.loss_terms = loss_terms;
    p.dlogits = dlogits;
    p.dvalues = dvalues;
    p.vtarget = vtarget;
    p.advantage = advantage;
    p.partials = static_cast<float*>(workspace);
    p.counter = reinterpret_cast<unsigned int*>(static_cast<char*>(workspace) +
                                                (size_t)kMaxGridBlocks * 8 * sizeof(float));
    p.tagged_rows = reinterpret_cast<unsigned long long*>(static_cast<char*>(workspace) +
                                                          (size_t)kMaxGridBlocks * 8 * sizeof(float) + kCounterBytes);
    // room for the tiles' aggregates is optional: without it long trajectories are swept inside one block
    p.tile_aggregates = (T > kMinTileRows && workspace_bytes >= impact_loss_workspace_bytes(B, T))
                            ? reinterpret_cast<unsigned long long*>(static_cast<char*>(workspace) + kWorkspaceFixedBytes)
                            : nullptr;
    p.target_copy = target_logits_copy;
    p.indirect = indirect;
    p.A = A;
    return run_categorical(p, B, T, logits_dtype == IMPACT_DTYPE_BF16, coef->dlogits_dtype == IMPACT_DTYPE_BF16,
                           di, static_cast<cudaStream_t>(stream));
}

extern "C" int32_t impact_loss_fwd_bwd(
    const void* learner_logits, const void* target_logits, const float* worker_logp,
    const int32_t* actions, const float* rewards, const float* discounts, const float* values,
    const float* bootstrap_values, float rho_bar, float c_bar, float clip_eps,
    const impact_coefficients* coef, int64_t B, int64_t T, int32_t A, int32_t logits_dtype,
    float* loss_terms, void* dlogits, float* dvalues, float* vtarget, float* advantage,
    void* workspace, size_t workspace_bytes, void* stream) {
    return loss_fwd_bwd_impl(learner_logits, target_logits, worker_logp, actions, rewards, discounts, values,
                             bootstrap_values, rho_bar, c_bar, clip_eps, coef, B, T, A, logits_dtype, loss_terms,
                             dlogits, dvalues, vtarget, advantage, workspace, workspace_bytes, nullptr, nullptr, stream);
}

extern "C" int32_t impact_loss_fwd_bwd_call(const impact_loss_call* c, void* stream) {
    if (!c) return IMPACT_ERR_INVALID_ARG;
    return loss_fwd_bwd_impl(c->learner_logits, c->target_logits, c->worker_logp, c->actions, c->rewards,
                             c->discounts, c->values, c->bootstrap_values, c->rho_bar, c->c_bar, c->clip_eps,
                             &c->coef, c->B, c->T, c->A, c->logits_dtype, c->loss_terms, c->dlogits,
                             c->dvalues, c->vtarget, c->advantage, c->workspace, c->workspace_bytes,
                             c->target_logits_copy, c->inputs_on_device, stream);
}

extern "C" int32_t impact_loss_fwd_bwd_gaussian(
    const float* learner_mean, const float* learner_logstd, const float* target_mean,
    const float* target_logstd, const float* worker_logp, const float* actions,
    const float* rewards, const float* discounts, const float* values,
    const float* bootstrap_values, float rho_bar, float c_bar, float clip_eps,
    const impact_coefficients* coef, int64_t B, int64_t T, int32_t D,
    float* loss_terms, float* dmean, float* dlogstd, float* dvalues, float* vtarget,
    float* advantage, void* workspace, size_t workspace_bytes, void* stream) {
    if (!learner_mean || !learner_logstd || !target_mean || !target_logstd || !worker_logp ||
        !actions || !rewards || !discounts || !values || !bootstrap_values || !coef || !loss_terms ||
        !dmean || !dlogstd || !dvalues || !workspace)
        return IMPACT_ERR_INVALID_ARG;
    if (B <= 0 || T <= 0 || D <= 0) return IMPACT_ERR_INVALID_ARG;
    const void* ptrs[] = {learner_mean, learner_logstd, target_mean, target_logstd, worker_logp,
                          actions, rewards, discounts, values, bootstrap_values, loss_terms,
                          dmean, dlogstd, dvalues, workspace};
    for (const void* q : ptrs)
        if (!aligned16(q)) return IMPACT_ERR_INVALID_ARG;
    if ((vtarget && !aligned16(vtarget)) || (advantage && !aligned16(advantage))) return IMPACT_ERR_INVALID_ARG;
    if (coef->dlogits_dtype != IMPACT_DTYPE_F32) return IMPACT_ERR_INVALID_ARG;
    if (D > 256) return IMPACT_ERR_UNSUPPORTED;
    if ((double)B * (double)T * (double)D >= 1099511627776.0 || (double)B * (double)T >= 4.0e12)
        return IMPACT_ERR_UNSUPPORTED;
    if (workspace_bytes < kWorkspaceFixedBytes) return IMPACT_ERR_WORKSPACE_TOO_SMALL;

    GaussParams p;
    int32_t st = fill_scalars(p.k, rho_bar, c_bar, clip_eps, coef, B, T);
    if (st != IMPACT_OK) return st;
    const DeviceInfo* di = current_device_info();
    if (!di) return IMPACT_ERR_CUDA;

    p.learner_mean = learner_mean;
    p.learner_logstd = learner_logstd;
    p.target_mean = target_mean;
    p.target_logstd = target_logstd;
    p.actions = actions;
    p.worker_logp = worker_logp;
    p.rewards = rewards;
    p.discounts = discounts;
    p.values = values;
    p.bootstrap = bootstrap_values;
    p.loss_terms = loss_terms;
    p.dmean = dmean;
    p.dlogstd = dlogstd;
    p.dvalues = dvalues;
    p.vtarget = vtarget;
    p.advantage = advantage;
    p.partials = static_cast<float*>(workspace);
    p.counter = reinterpret_cast<unsigned int*>(static_cast<char*>(workspace) +
                                                (size_t)kMaxGridBlocks * 8 * sizeof(float));
    p.tagged_rows = reinterpret_cast<unsigned long long*>(static_cast<char*>(workspace) +
                                                          (size_t)kMaxGridBlocks * 8 * sizeof(float) + kCounterBytes);
    p.tile_aggregates = (T > kRegTileRows && workspace_bytes >= impact_loss_workspace_bytes(B, T))
                            ? reinterpret_cast<unsigned long long*>(static_cast<char*>(workspace) + kWorkspaceFixedBytes)
                            : nullptr;
    p.D = D;
    if (has_gaussian_reg_kernel(D)) {
        p.Ds = D;
        p.geo = make_geometry(B, T, kRegTileRows);
        cudaStream_t rs = static_cast<cudaStream_t>(stream);
        switch (D) {
            case 3: return launch_gaussian_reg<3>(p, di, rs);
            case 6: return launch_gaussian_reg<6>(p, di, rs);
            default: return launch_gaussian_reg<17>(p, di, rs);
        }
    }
    p.Ds = pad_odd(D);
    const int nt = pick_nt(p.Ds, 5, 100 * 1024);
    p.geo = make_geometry(B, T, nt);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (nt) {
        case 128: return launch_gaussian<128>(p, di, s);
        case 64: return launch_gaussian<64>(p, di, s);
        default: return launch_gaussian<32>(p, di, s);
    }
}

// ------------------------------------------------------------------------------------------
// Variant for callers that must not allocate
// ------------------------------------------------------------------------------------------
namespace impact {
namespace {

constexpr int kStaticMaxBlocks = 1024;  // tiles (= blocks) the built-in scratch has room for
constexpr size_t kStaticScratchBytes = (size_t)kStaticMaxBlocks * 8 * sizeof(float) + kCounterBytes +
                                       (size_t)kMaxTaggedRows * 8 * sizeof(unsigned long long);

// Scratch that lives in the library image, laid out like a workspace: per-block sums, 256 bytes of
// counter words, the tagged rows of the persistent kernel.  Every device that loads the library
// carries its own copy.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of g_static_scratch on the current device.  In host code the symbol's name
// is only a handle, so the address is asked for once per device and remembered.
int32_t static_scratch_address(const DeviceInfo* di, unsigned char** out) {
    static unsigned char* address[64] = {};
    if (!address[di->device]) {
        void* p = nullptr;
        IMPACT_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        address[di->device] = static_cast<unsigned char*>(p);
    }
    *out = address[di->device];
    return IMPACT_OK;
}

}  // namespace
}  // namespace impact

extern "C" int32_t impact_loss_fwd_bwd_static_scratch(
    const void* learner_logits, const void* target_logits, const float* worker_logp,
    const int32_t* actions, const float* rewards, const float* discounts, const float* values,
    const float* bootstrap_values, float rho_bar, float c_bar, float clip_eps,
    const impact_coefficients* coef, int64_t B, int64_t T, int32_t A, int32_t logits_dtype,
    float* loss_terms, void* dlogits, float* dvalues, float* vtarget, float* advantage,
    void* stream) {
    if (!learner_logits || !target_logits || !worker_logp || !actions || !rewards || !discounts ||
        !values || !bootstrap_values || !coef || !loss_terms || !dlogits || !dvalues)
        return IMPACT_ERR_INVALID_ARG;
    if (B <= 0 || T <= 0 || A <= 0) return IMPACT_ERR_INVALID_ARG;
    const void* ptrs[] = {learner_logits, target_logits, worker_logp, actions, rewards, discounts,
                          values, bootstrap_values, loss_terms, dlogits, dvalues};
    for (const void* q : ptrs)
        if (!aligned16(q)) return IMPACT_ERR_INVALID_ARG;
    if ((vtarget && !aligned16(vtarget)) || (advantage && !aligned16(advantage))) return IMPACT_ERR_INVALID_ARG;
    if (logits_dtype != IMPACT_DTYPE_F32 && logits_dtype != IMPACT_DTYPE_BF16) return IMPACT_ERR_INVALID_ARG;
    if (coef->dlogits_dtype != IMPACT_DTYPE_F32 && coef->dlogits_dtype != IMPACT_DTYPE_BF16)
        return IMPACT_ERR_INVALID_ARG;
    if (A > 64) return IMPACT_ERR_UNSUPPORTED;  // keeps the tile at 64 steps or more, which the limit below counts in

    CatParams p = {};
    int32_t st = fill_scalars(p.k, rho_bar, c_bar, clip_eps, coef, B, T);
    if (st != IMPACT_OK) return st;
    p.A = A;
    // one block's sums per tile at most: more tiles than the built-in scratch holds are refused
    const bool logits_bf16 = logits_dtype == IMPACT_DTYPE_BF16, grads_bf16 = coef->dlogits_dtype == IMPACT_DTYPE_BF16;
    const int tile_rows_here = categorical_tile_rows(A, logits_bf16, grads_bf16, T > ws_tile_rows(A));  // no aggregates here
    if (make_geometry(B, T, tile_rows_here).nchunks > kStaticMaxBlocks) return IMPACT_ERR_WORKSPACE_TOO_SMALL;

    const DeviceInfo* di = current_device_info();
    if (!di) return IMPACT_ERR_CUDA;
    unsigned char* scratch = nullptr;
    st = static_scratch_address(di, &scratch);
    if (st != IMPACT_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the scratch keeps whatever the previous call left; the completion counter is what has to start at zero.  The
    // error word next to it stays as it is (it is sticky until impact_loss_static_scratch_status clears it), and so
    // does the launch number, which is what tells this call's rows from the previous call's.
    unsigned char* counter = scratch + (size_t)kStaticMaxBlocks * 8 * sizeof(float);
    IMPACT_CUDA_TRY(cudaMemsetAsync(counter, 0, sizeof(unsigned int), s));

    p.learner_logits = learner_logits;
    p.target_logits = target_logits;
    p.worker_logp = worker_logp;
    p.actions = actions;
    p.rewards = rewards;
    p.discounts = discounts;
    p.values = values;
    p.bootstrap = bootstrap_values;
    p.loss_terms = loss_terms;
    p.dlogits = dlogits;
    p.dvalues = dvalues;
    p.vtarget = vtarget;
    p.advantage = advantage;
    p.partials = reinterpret_cast<float*>(scratch);
    p.counter = reinterpret_cast<unsigned int*>(counter);
    p.tagged_rows = reinterpret_cast<unsigned long long*>(counter + kCounterBytes);
    p.tile_aggregates = nullptr;  // long trajectories are swept tile by tile inside a block
    p.target_copy = nullptr;
    // the same kernels, chosen the same way, as impact_loss_fwd_bwd
    return run_categorical(p, B, T, logits_dtype == IMPACT_DTYPE_BF16, coef->dlogits_dtype == IMPACT_DTYPE_BF16,
                           di, s);
}

extern "C" int32_t impact_loss_static_scratch_status(int32_t* flag_out, int32_t clear, void* stream) {
    if (!flag_out) return IMPACT_ERR_INVALID_ARG;
    const DeviceInfo* di = current_device_info();
    if (!di) return IMPACT_ERR_CUDA;
    unsigned char* scratch = nullptr;
    const int32_t st = static_scratch_address(di, &scratch);
    if (st != IMPACT_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned char* word = scratch + (size_t)kStaticMaxBlocks * 8 * sizeof(float) + sizeof(unsigned int);
    unsigned int flag = 0;
    IMPACT_CUDA_TRY(cudaMemcpyAsync(&flag, word, sizeof(flag), cudaMemcpyDeviceToHost, s));
    IMPACT_CUDA_TRY(cudaStreamSynchronize(s));
    if (clear && flag != 0) IMPACT_CUDA_TRY(cudaMemsetAsync(word, 0, sizeof(unsigned int), s));
    *flag_out = (int32_t)flag;
    return IMPACT_OK;
}
