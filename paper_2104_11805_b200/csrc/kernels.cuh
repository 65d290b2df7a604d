// Device kernels of the sparse-DNN SGD hot path (sm_100a).
//
// Data layout.  Activations, deltas and the partial products S = W^T delta live in
// neuron-major tiles X[i*ld + b] (neuron i, input b; ld = padded batch, a multiple of 4),
// so that the row of X gathered for one stored entry W(i,j) is contiguous and every
// access is a 128-bit vector.  A row of a tile is shared by G lanes (G*4 batch entries,
// one float4 per lane); a warp therefore works on 32/G matrix rows at once.  Tiles
// wider than 128 inputs are processed in chunks of 128 (blockIdx.y).
//
// Equations (paper, Section 3.2): forward x^k = f(W^k x^{k-1} + b^k); recursion
// delta^{k-1} = (W^k)^T delta^k (.) f'(z^{k-1}); update W^k(j,i) -= eta delta^k(j) x^{k-1}(i)
// on stored entries.  Only x^k is stored: with f = clamp to [0,c], f'(z) = [0 < x < c].
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace sdnn_kernels {

struct StepParams {     // written by set_step_params before each train step; read by the graph's kernels
    float eta;          // learning rate
    float inv_b;        // 1 / B
    int   batch;        // B (valid inputs; the tile is zero-padded to ld)
    int   pad;
};

__device__ __forceinline__ float4 ld_f4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ void st_f4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }

// read-only gather of a tile row segment (goes through the non-coherent path)
__device__ __forceinline__ float4 gather_f4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }

// 128-bit vector reduction into global memory (sm_90+): four fp32 adds in one L2 operation
__device__ __forceinline__ void red_add_f4(float* p, float4 v) {
    asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                 :: "l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}

__device__ __forceinline__ float clampf(float z, float c) { return fminf(fmaxf(z, 0.0f), c); }
__device__ __forceinline__ float dmask(float x, float c) { return (x > 0.0f && x < c) ? 1.0f : 0.0f; }

// sum over the G lanes of a row group; `gmask` names exactly those lanes, so that groups of one warp
// whose rows have different lengths may sit in different loop iterations
template <int G>
__device__ __forceinline__ float group_sum(float v, unsigned gmask) {
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) v += __shfl_xor_sync(gmask, v, o);
    return v;
}

// ---------------------------------------------------------------------------------------------
// x0 [cnt][n] (input-major, as the caller passes it)  ->  tile [n][ld], zero-padded for b >= cnt.
// Block (32, 8); grid (ceil(n/32), ceil(cols/32)) where cols = padded columns to fill.
__global__ void transpose_in_kernel(const float* __restrict__ src, float* __restrict__ dst,
                                    int n, int cnt, int cols, int ld) {
    __shared__ float t[32][33];
    const int i0 = blockIdx.x * 32, b0 = blockIdx.y * 32;
    for (int r = threadIdx.y; r < 32; r += 8) {
        int b = b0 + r, i = i0 + threadIdx.x;
        t[r][threadIdx.x] = (b < cnt && i < n) ? src[(size_t)b * n + i] : 0.0f;
    }
    __syncthreads();
    for (int r = threadIdx.y; r < 32; r += 8) {
        int i = i0 + r, b = b0 + threadIdx.x;
        if (i < n && b < cols) dst[(size_t)i * ld + b] = t[threadIdx.x][r];
    }
}

// tile [n][ld] -> y [cnt][n]
__global__ void transpose_out_kernel(const float* __restrict__ src, float* __restrict__ dst,
                                     int n, int cnt, int ld) {
    __shared__ float t[32][33];
    const int i0 = blockIdx.x * 32, b0 = blockIdx.y * 32;
    for (int r = threadIdx.y; r < 32; r += 8) {
        int i = i0 + r, b = b0 + threadIdx.x;
        t[r][threadIdx.x] = (i < n && b < cnt) ? src[(size_t)i * ld + b] : 0.0f;
    }
    __syncthreads();
    for (int r = threadIdx.y; r < 32; r += 8) {
        int b = b0 + r, i = i0 + threadIdx.x;
        if (b < cnt && i < n) dst[(size_t)b * n + i] = t[threadIdx.x][r];
    }
}

__global__ void set_step_params_kernel(StepParams* p, float eta, int batch, double* loss) {
    p->eta = eta; p->inv_b = 1.0f / (float)batch; p->batch = batch; p->pad = 0;
    *loss = 0.0;
}

// ---------------------------------------------------------------------------------------------
// Forward layer (feedforward equation): Xout[i,:] = clamp(bias[i] + sum_p val[p] * Xin[col[p],:]).
// One group of G lanes per matrix row; each lane accumulates 4 batch entries.  The products of a
// row are added in CSR order with fp32 FMAs.  Index/value loads are 128-bit when the row segment
// is 16-byte aligned (always the case for rows of 4k entries in a 16-byte aligned layer).
template <int G>
__global__ void __launch_bounds__(256)
forward_kernel(const int* __restrict__ row_ptr, const int* __restrict__ col, const float* __restrict__ val,
               const float* __restrict__ bias, const float* __restrict__ xin, float* __restrict__ xout,
               int n, int ld, float clamp) {
    constexpr int RPW = 32 / G;
    const int lane = threadIdx.x & 31;
    const int sub = lane % G, grp = lane / G;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int row = warp * RPW + grp;
    if (row >= n) return;
    const int boff = blockIdx.y * (4 * G) + sub * 4;
    const float* xg = xin + boff;

    const int s = row_ptr[row], e = row_ptr[row + 1];
    const float b = bias[row];
    float4 acc = make_float4(b, b, b, b);
    int p = s;
    if (((s | e) & 3) == 0) {
        for (; p + 8 <= e; p += 8) {
            const int4 c0 = *reinterpret_cast<const int4*>(col + p), c1 = *reinterpret_cast<const int4*>(col + p + 4);
            const float4 w0 = ld_f4(val + p), w1 = ld_f4(val + p + 4);
            const float4 x0 = gather_f4(xg + (size_t)c0.x * ld), x1 = gather_f4(xg + (size_t)c0.y * ld);
            const float4 x2 = gather_f4(xg + (size_t)c0.z * ld), x3 = gather_f4(xg + (size_t)c0.w * ld);
            const float4 x4 = gather_f4(xg + (size_t)c1.x * ld), x5 = gather_f4(xg + (size_t)c1.y * ld);
            const float4 x6 = gather_f4(xg + (size_t)c1.z * ld), x7 = gather_f4(xg + (size_t)c1.w * ld);
#define SDNN_FMA4(W, X) acc.x = fmaf(W, X.x, acc.x); acc.y = fmaf(W, X.y, acc.y); acc.z = fmaf(W, X.z, acc.z); acc.w = fmaf(W, X.w, acc.w);
            SDNN_FMA4(w0.x, x0) SDNN_FMA4(w0.y, x1) SDNN_FMA4(w0.z, x2) SDNN_FMA4(w0.w, x3)
            SDNN_FMA4(w1.x, x4) SDNN_FMA4(w1.y, x5) SDNN_FMA4(w1.z, x6) SDNN_FMA4(w1.w, x7)
        }
        for (; p < e; p += 4) {
            const int4 c0 = *reinterpret_cast<const int4*>(col + p);
            const float4 w0 = ld_f4(val + p);
            const float4 x0 = gather_f4(xg + (size_t)c0.x * ld), x1 = gather_f4(xg + (size_t)c0.y * ld);
            const float4 x2 = gather_f4(xg + (size_t)c0.z * ld), x3 = gather_f4(xg + (size_t)c0.w * ld);
            SDNN_FMA4(w0.x, x0) SDNN_FMA4(w0.y, x1) SDNN_FMA4(w0.z, x2) SDNN_FMA4(w0.w, x3)
        }
    } else {
        for (; p < e; ++p) {
            const float w = val[p];
            const float4 x = gather_f4(xg + (size_t)col[p] * ld);
            SDNN_FMA4(w, x)
        }
    }
    acc.x = clampf(acc.x, clamp); acc.y = clampf(acc.y, clamp);
    acc.z = clampf(acc.z, clamp); acc.w = clampf(acc.w, clamp);
    st_f4(xout + (size_t)row * ld + boff, acc);
}

// ---------------------------------------------------------------------------------------------
// Backward + update of one layer k in ONE pass over its stored entries (Algorithm 1, loop body):
//   delta^k[i,:]   = LAST ? (x^L[i,:] - y[i,:]) (.) f'   :  S_k[i,:] (.) f'      with f' = [0 < x^k < c]
//   for each stored (i,j), old weight w:
//       g          = sum_b delta^k[i,b] x^{k-1}[j,b]                 (masked gradient, times B)
//       S_{k-1}[j,:] += w * delta^k[i,:]      (PROP; w is the value BEFORE the update)
//       W(i,j)     = w - (eta/B) g
// S_k is cleared row by row as it is consumed, so the two S buffers can alternate between layers
// without a separate memset.  The scatter uses one 128-bit vector reduction per lane.  The whole
// minibatch sits in one chunk (ld = 4G <= 128), so each weight is owned by exactly one lane group.
template <int G, bool LAST, bool PROP>
__global__ void __launch_bounds__(256)
backward_kernel(const int* __restrict__ row_ptr, const int* __restrict__ col, float* __restrict__ val,
                float* __restrict__ bias, const float* __restrict__ xk, const float* __restrict__ xprev,
                float* __restrict__ s_k /* LAST: target tile y */, float* __restrict__ s_prev,
                int n, float clamp, const StepParams* __restrict__ sp, double* __restrict__ loss,
                float* __restrict__ dbg_delta, float* __restrict__ dbg_grad, int update_bias, int skip_dead) {
    constexpr int RPW = 32 / G;
    constexpr int ld = 4 * G;
    const int lane = threadIdx.x & 31;
    const int sub = lane % G, grp = lane / G;
    const unsigned gmask = (G == 32) ? 0xffffffffu : (((1u << G) - 1u) << (grp * G));
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int row = warp * RPW + grp;
    const int boff = sub * 4;
    const float inv_b = sp->inv_b;
    const float step = sp->eta * inv_b;
    const bool valid = row < n;

    float4 d = make_float4(0.f, 0.f, 0.f, 0.f);
    float sq = 0.0f;
    if (valid) {
        const size_t o = (size_t)row * ld + boff;
        const float4 x = ld_f4(xk + o);
        float4 t = ld_f4(s_k + o);
        if (LAST) {
            const int nb = sp->batch;
            t.x = (boff + 0 < nb) ? x.x - t.x : 0.0f; t.y = (boff + 1 < nb) ? x.y - t.y : 0.0f;
            t.z = (boff + 2 < nb) ? x.z - t.z : 0.0f; t.w = (boff + 3 < nb) ? x.w - t.w : 0.0f;
            sq = t.x * t.x + t.y * t.y + t.z * t.z + t.w * t.w;
        } else {
            st_f4(s_k + o, make_float4(0.f, 0.f, 0.f, 0.f));
        }
        d.x = t.x * dmask(x.x, clamp); d.y = t.y * dmask(x.y, clamp);
        d.z = t.z * dmask(x.z, clamp); d.w = t.w * dmask(x.w, clamp);
        if (dbg_delta) st_f4(dbg_delta + o, d);
    }
    if (LAST) {   // loss J = 1/(2B) sum (x^L - y)^2 : block sum in fp32 partials, one double atomic per block
        __shared__ float part[8];
        float w = sq;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) w += __shfl_xor_sync(0xffffffffu, w, o);
        if (lane == 0) part[threadIdx.x >> 5] = w;
        __syncthreads();
        if (threadIdx.x == 0) {
            double tot = 0.0;
            for (int q = 0; q < (int)(blockDim.x >> 5); ++q) tot += (double)part[q];
            if (tot != 0.0) atomicAdd(loss, 0.5 * tot * (double)inv_b);
        }
    }
    if (!valid) return;      // whole groups leave together; the shuffles below name only the group's lanes
    if (update_bias) {       // bias read as one more column of W^k whose input is the constant 1
        const float bg = group_sum<G>(d.x + d.y + d.z + d.w, gmask);
        if (sub == 0) bias[row] -= step * bg;
    }
    if (skip_dead) {
        const bool alive = !(d.x == 0.0f && d.y == 0.0f && d.z == 0.0f && d.w == 0.0f);
        if ((__ballot_sync(gmask, alive) & gmask) == 0u) return;   // delta^k(i) = 0 for every input: nothing changes
    }

    const float* xg = xprev + boff;
    float* sg = s_prev + boff;
    const int s = row_ptr[row], e = row_ptr[row + 1];
    int p = s;
#define SDNN_DOT4(X) fmaf(d.w, X.w, fmaf(d.z, X.z, fmaf(d.y, X.y, d.x * X.x)))
#define SDNN_SCAT(C, W) red_add_f4(sg + (size_t)(C) * ld, make_float4(W * d.x, W * d.y, W * d.z, W * d.w));
    if (((s | e) & 3) == 0) {
        for (; p < e; p += 4) {
            const int4 c = *reinterpret_cast<const int4*>(col + p);
            const float4 w = ld_f4(val + p);
            const float4 x0 = gather_f4(xg + (size_t)c.x * ld), x1 = gather_f4(xg + (size_t)c.y * ld);
            const float4 x2 = gather_f4(xg + (size_t)c.z * ld), x3 = gather_f4(xg + (size_t)c.w * ld);
            if (PROP) { SDNN_SCAT(c.x, w.x) SDNN_SCAT(c.y, w.y) SDNN_SCAT(c.z, w.z) SDNN_SCAT(c.w, w.w) }
            float4 g;
            g.x = group_sum<G>(SDNN_DOT4(x0), gmask); g.y = group_sum<G>(SDNN_DOT4(x1), gmask);
            g.z = group_sum<G>(SDNN_DOT4(x2), gmask); g.w = group_sum<G>(SDNN_DOT4(x3), gmask);
            if (sub == 0) {
                st_f4(val + p, make_float4(fmaf(-step, g.x, w.x), fmaf(-step, g.y, w.y),
                                           fmaf(-step, g.z, w.z), fmaf(-step, g.w, w.w)));
                if (dbg_grad) st_f4(dbg_grad + p, make_float4(g.x * inv_b, g.y * inv_b, g.z * inv_b, g.w * inv_b));
            }
        }
    } else {
        for (; p < e; ++p) {
            const int c = col[p];
            const float w = val[p];
            const float4 x = gather_f4(xg + (size_t)c * ld);
            if (PROP) { SDNN_SCAT(c, w) }
            const float g = group_sum<G>(SDNN_DOT4(x), gmask);
            if (sub == 0) {
                val[p] = fmaf(-step, g, w);
                if (dbg_grad) dbg_grad[p] = g * inv_b;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Final-layer nonzero sets.  The tile is cut into segments of SEG rows.
//   count: seg_cnt[seg*ld + b] = #{ i in segment : X[i,b] != 0 }
//   scan : per input b: nz_count[b] = total; seg_cnt becomes the exclusive prefix over segments
//   offs : exclusive scan of nz_count over the inputs of the tile, added to the running total
//   fill : ids written in ascending order at offs[b] + prefix[seg][b]
constexpr int NZ_SEG = 256;

__global__ void nz_count_kernel(const float* __restrict__ x, int* __restrict__ seg_cnt, int n, int cnt, int ld) {
    const int b = blockIdx.y * blockDim.x + threadIdx.x;
    if (b >= cnt) return;
    const int i0 = blockIdx.x * NZ_SEG, i1 = min(n, i0 + NZ_SEG);
    int c = 0;
    for (int i = i0; i < i1; ++i) c += (x[(size_t)i * ld + b] != 0.0f);
    seg_cnt[(size_t)blockIdx.x * ld + b] = c;
}

__global__ void nz_scan_segments_kernel(int* __restrict__ seg_cnt, int* __restrict__ tile_cnt, int nseg, int cnt, int ld) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= cnt) return;
    int run = 0;
    for (int sgm = 0; sgm < nseg; ++sgm) {
        int c = seg_cnt[(size_t)sgm * ld + b];
        seg_cnt[(size_t)sgm * ld + b] = run;
        run += c;
    }
    tile_cnt[b] = run;
}

// single block of 1024 threads: offs[b] = running + exclusive_scan(tile_cnt)[b]; running += total
__global__ void nz_scan_inputs_kernel(const int* __restrict__ tile_cnt, long long* __restrict__ offs,
                                      long long* __restrict__ running, int* __restrict__ count_out, int cnt) {
    __shared__ long long warp_tot[32];
    __shared__ long long carry;
    if (threadIdx.x == 0) carry = *running;
    __syncthreads();
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (int base = 0; base < cnt; base += 1024) {
        const int b = base + threadIdx.x;
        const long long v = (b < cnt) ? tile_cnt[b] : 0;
        long long incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            long long t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) warp_tot[wid] = incl;
        __syncthreads();
        if (wid == 0) {
            long long w = warp_tot[lane], wi = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                long long t = __shfl_up_sync(0xffffffffu, wi, o);
                if (lane >= o) wi += t;
            }
            warp_tot[lane] = wi - w;   // exclusive prefix of the warp totals
        }
        __syncthreads();
        const long long excl = carry + warp_tot[wid] + incl - v;
        if (b < cnt) {
            offs[b] = excl;
            if (count_out) count_out[b] = (int)v;
        }
        __syncthreads();
        if (threadIdx.x == 1023) carry = excl + v;
        __syncthreads();
    }
    if (threadIdx.x == 0) *running = carry;
}

__global__ void nz_fill_kernel(const float* __restrict__ x, const int* __restrict__ seg_pre,
                               const long long* __restrict__ offs, int* __restrict__ out, long long capacity,
                               int n, int cnt, int ld) {
    const int b = blockIdx.y * blockDim.x + threadIdx.x;
    if (b >= cnt) return;
    const int i0 = blockIdx.x * NZ_SEG, i1 = min(n, i0 + NZ_SEG);
    long long pos = offs[b] + seg_pre[(size_t)blockIdx.x * ld + b];
    for (int i = i0; i < i1; ++i) {
        if (x[(size_t)i * ld + b] != 0.0f) {
            if (pos < capacity) out[pos] = i;
            ++pos;
        }
    }
}

}  // namespace sdnn_kernels
