// Backward pass of one SwitchHead layer, fp32 configuration, CUDA cores.
//
// The paper gives no backward formulas (its training relies on automatic differentiation of the forward
// equations of Sec. 2.2); these kernels are the chain rule for those equations with the expert selection
// held fixed (top-k is piecewise constant).  Given G = dL/dy and the intermediates the forward pass left
// in the workspace (Q - stored times log2(e)/sqrt(d_head) -, K, V as [B, H, T, D]; Ahat as [N, H, D]; the
// selections and gates of both sides):
//   output experts   dsD[t,h,j] = (Ahat[t,h] W_O^{h,e}) . G[t];  dAhat[t,h] += sD (W_O^{h,e} G[t]);  dW_O^{h,e} += sD Ahat[t,h]^T G[t]
//   attention        dV = A^T dAhat;  dS = A o (dAhat V^T - rowsum(dAhat o Ahat));  dQ = dS K / sqrt(d);  dK = dS^T Q / sqrt(d)
//   value experts    dsS[t,h,j] = (x[t] W_V^{h,e}) . dV[t,h];  dx[t] += sS (W_V^{h,e} dV[t,h]);  dW_V^{h,e} += sS x[t]^T dV[t,h]
//   dense Q, K       dx += dQ W_Q^T + dK W_K^T;  dW_Q = x^T dQ;  dW_K = x^T dK
//   gates            dz = ds s (1 - s) at the selected entries;  dx += dz W^T;  dW = x^T dz     (both sides)
// Plain kernels, one block per (token, head) or per token, sums over tokens by fp32 atomics: this path
// serves the small fp32 configuration (exact-arithmetic parity with the oracle), not throughput.
// Weight copies in the workspace (fp32): wqk [(which*H + h)*D + dd][m], wv [(h*E + e)*D + dd][m],
// wo [(h*E + e)*M + m][dd], wgate [(side*H + h)*E + e][m]; gradients go out in the layouts the weights
// were given in (d_head unpadded).
#pragma once
#include "sh_internal.cuh"

struct ShBwArgs {
  ShDims d;
  const float* x;            // [N, M]
  const float* dy;           // [N, M]
  const float *q, *k, *v;    // [B, H, T, D]
  const float* ahat;         // [N, H, D]
  const int* idx;            // [2, N, H, k]
  const float* gate;         // [2, N, H, k]
  const float *wqk, *wv, *wo, *wgate;
  float *dq, *dk, *dv, *dahat;     // [N, H, D] scratch (token-major)
  float* dgate;              // [2, N, H, k] scratch
  float *dx, *dWq, *dWk, *dWv, *dWo, *dWs, *dWd;
};

static __device__ __forceinline__ float sh_block_sum(float v, float* red) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];
  return t;
}

// Output experts.  Block = (token t, head h), 128 threads.
static __global__ void __launch_bounds__(128) sh_bw_o_kernel(ShBwArgs a) {
  const ShDims& d = a.d;
  __shared__ float s_w[256], s_ah[256], red[4];
  const int t = blockIdx.x / d.H, h = blockIdx.x % d.H;
  const float* dy = a.dy + (size_t)t * d.M;
  const float* ah = a.ahat + ((size_t)t * d.H + h) * d.D;
  for (int dd = threadIdx.x; dd < d.D; dd += blockDim.x) s_ah[dd] = ah[dd];
  float acc[2] = {0.f, 0.f};                                // dAhat for dd = tid, tid + 128
  for (int j = 0; j < d.k; ++j) {
    const size_t so = (((size_t)1 * d.N + t) * d.H + h) * d.k + j;   // destination side
    const int e = a.idx[so];
    const float g = a.gate[so];
    const float* W = a.wo + (size_t)(h * d.E + e) * d.M * d.D;        // [m][dd]
    __syncthreads();
    for (int dd = threadIdx.x; dd < d.D; dd += blockDim.x) {
      float w = 0.f;
      for (int m = 0; m < d.M; ++m) w = fmaf(W[(size_t)m * d.D + dd], dy[m], w);
      s_w[dd] = w;
      acc[dd / 128] = fmaf(g, w, acc[dd / 128]);
    }
    float part = 0.f;
    __syncthreads();
    for (int dd = threadIdx.x; dd < d.D; dd += blockDim.x) part = fmaf(s_ah[dd], s_w[dd], part);
    const float dg = sh_block_sum(part, red);
    if (threadIdx.x == 0) a.dgate[so] = dg;
    float* dW = a.dWo + (size_t)(h * d.E + e) * d.Dt * d.M;           // [dd][m], dd < Dt
    for (int i = threadIdx.x; i < d.Dt * d.M; i += blockDim.x) {
      const int dd = i / d.M, m = i % d.M;
      atomicAdd(dW + i, g * s_ah[dd] * dy[m]);
    }
  }
  float* da = a.dahat + ((size_t)t * d.H + h) * d.D;
  for (int dd = threadIdx.x; dd < d.D; dd += blockDim.x) da[dd] = acc[dd / 128];
}

// Attention.  One warp per query row (b, h, i); lane = features lane, lane + 32, ...
static __global__ void __launch_bounds__(128) sh_bw_attn_kernel(ShBwArgs a) {
  const ShDims& d = a.d;
  const long row = ((long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (row >= (long)d.B * d.H * d.T) return;
  const int i = (int)(row % d.T), h = (int)((row / d.T) % d.H), b = (int)(row / ((long)d.T * d.H));
  const int NR = d.D / 32;                                   // features per lane (1..8)
  const float* qrow = a.q + (((size_t)b * d.H + h) * d.T + i) * d.D;
  const float* kbase = a.k + ((size_t)b * d.H + h) * d.T * d.D;
  const float* vbase = a.v + ((size_t)b * d.H + h) * d.T * d.D;
  const size_t tok = (size_t)b * d.T + i;
  const float* dah = a.dahat + (tok * d.H + h) * d.D;
  const float* ah = a.ahat + (tok * d.H + h) * d.D;
  float qv[8], dav[8], dqv[8];
  float dsum = 0.f;
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    qv[r] = dav[r] = dqv[r] = 0.f;
    if (r < NR) { qv[r] = qrow[lane + 32 * r]; dav[r] = dah[lane + 32 * r]; dsum = fmaf(dav[r], ah[lane + 32 * r], dsum); }
  }
  for (int o = 16; o > 0; o >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, o);
  const int last = d.causal ? i : d.T - 1;
  // pass 1: maximum and normaliser of the row (scores in base-2 units: Q carries log2(e)/sqrt(d_head))
  float m2 = -INFINITY, l = 0.f;
  for (int j = 0; j <= last; ++j) {
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < 8; ++r) if (r < NR) s = fmaf(qv[r], kbase[(size_t)j * d.D + lane + 32 * r], s);
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const float mn = fmaxf(m2, s);
    l = l * exp2f(m2 - mn) + exp2f(s - mn);
    m2 = mn;
  }
  const float inv_sqrt_d = rsqrtf((float)d.Dt);
  const float k_scale = 0.6931471805599453f;                 // dK = dS Q_real / sqrt(d) = dS Q_stored / log2(e)
  for (int j = 0; j <= last; ++j) {
    float s = 0.f, da = 0.f;
#pragma unroll
    for (int r = 0; r < 8; ++r)
      if (r < NR) {
        s = fmaf(qv[r], kbase[(size_t)j * d.D + lane + 32 * r], s);
        da = fmaf(dav[r], vbase[(size_t)j * d.D + lane + 32 * r], da);
      }
    for (int o = 16; o > 0; o >>= 1) { s += __shfl_xor_sync(0xffffffffu, s, o); da += __shfl_xor_sync(0xffffffffu, da, o); }
    const float p = exp2f(s - m2) / l;
    const float ds = p * (da - dsum);
    const size_t tj = ((size_t)b * d.T + j) * d.H + h;
#pragma unroll
    for (int r = 0; r < 8; ++r)
      if (r < NR) {
        const int dd = lane + 32 * r;
        dqv[r] = fmaf(ds, kbase[(size_t)j * d.D + dd], dqv[r]);
        atomicAdd(a.dk + tj * d.D + dd, ds * qv[r] * k_scale);
        atomicAdd(a.dv + tj * d.D + dd, p * dav[r]);
      }
  }
#pragma unroll
  for (int r = 0; r < 8; ++r)
    if (r < NR) a.dq[(tok * d.H + h) * d.D + lane + 32 * r] = dqv[r] * inv_sqrt_d;
}

// Value experts.  Block = (token t, head h), 128 threads over d_model.
static __global__ void __launch_bounds__(128) sh_bw_v_kernel(ShBwArgs a) {
  const ShDims& d = a.d;
  __shared__ float s_dv[256], red[4];
  const int t = blockIdx.x / d.H, h = blockIdx.x % d.H;
  const float* x = a.x + (size_t)t * d.M;
  const float* dv = a.dv + ((size_t)t * d.H + h) * d.D;
  for (int dd = threadIdx.x; dd < d.D; dd += blockDim.x) s_dv[dd] = dv[dd];
  __syncthreads();
  for (int j = 0; j < d.k; ++j) {
    const size_t so = (((size_t)0 * d.N + t) * d.H + h) * d.k + j;   // source side
    const int e = a.idx[so];
    const float g = a.gate[so];
    const float* W = a.wv + (size_t)(h * d.E + e) * d.D * d.M;        // [dd][m]
    float part = 0.f;
    for (int m = threadIdx.x; m < d.M; m += blockDim.x) {
      float r = 0.f;
      for (int dd = 0; dd < d.D; ++dd) r = fmaf(W[(size_t)dd * d.M + m], s_dv[dd], r);
      part = fmaf(x[m], r, part);
      atomicAdd(a.dx + (size_t)t * d.M + m, g * r);
    }
    const float dg = sh_block_sum(part, red);
    if (threadIdx.x == 0) a.dgate[so] = dg;
    float* dW = a.dWv + (size_t)(h * d.E + e) * d.M * d.Dt;           // [m][dd], dd < Dt
    for (int i = threadIdx.x; i < d.M * d.Dt; i += blockDim.x) {
      const int m = i / d.Dt, dd = i % d.Dt;
      atomicAdd(dW + i, g * x[m] * s_dv[dd]);
    }
  }
}

// Dense queries and keys.  Block = token t, 128 threads over d_model.
static __global__ void __launch_bounds__(128) sh_bw_qk_kernel(ShBwArgs a) {
  const ShDims& d = a.d;
  extern __shared__ float s_g[];                            // [2][H * D]: dQ and dK of the token
  const int t = blockIdx.x;
  const int HD = d.H * d.D;
  const float* x = a.x + (size_t)t * d.M;
  for (int i = threadIdx.x; i < HD; i += blockDim.x) { s_g[i] = a.dq[(size_t)t * HD + i]; s_g[HD + i] = a.dk[(size_t)t * HD + i]; }
  __syncthreads();
  for (int m = threadIdx.x; m < d.M; m += blockDim.x) {
    float acc = 0.f;
    for (int i = 0; i < 2 * HD; ++i) acc = fmaf(s_g[i], a.wqk[(size_t)i * d.M + m], acc);   // rows (which*H + h)*D + dd = i
    atomicAdd(a.dx + (size_t)t * d.M + m, acc);
  }
  for (int which = 0; which < 2; ++which) {
    float* dW = which == 0 ? a.dWq : a.dWk;                  // [H][M][Dt]
    for (int i = threadIdx.x; i < d.H * d.M * d.Dt; i += blockDim.x) {
      const int dd = i % d.Dt, m = (i / d.Dt) % d.M, h = i / (d.Dt * d.M);
      atomicAdd(dW + i, x[m] * s_g[which * HD + h * d.D + dd]);
    }
  }
}

// Gates of both sides.  Block = token t, 128 threads over d_model.
static __global__ void __launch_bounds__(128) sh_bw_gate_kernel(ShBwArgs a) {
  const ShDims& d = a.d;
  const int t = blockIdx.x;
  const float* x = a.x + (size_t)t * d.M;
  for (int side = 0; side < 2; ++side) {
    float* dW = side == 0 ? a.dWs : a.dWd;                   // [H][M][E]
    for (int h = 0; h < d.H; ++h)
      for (int j = 0; j < d.k; ++j) {
        const size_t so = (((size_t)side * d.N + t) * d.H + h) * d.k + j;
        const int e = a.idx[so];
        const float g = a.gate[so];
        const float dz = a.dgate[so] * g * (1.f - g);
        const float* W = a.wgate + (size_t)((side * d.H + h) * d.E + e) * d.M;
        for (int m = threadIdx.x; m < d.M; m += blockDim.x) {
          atomicAdd(a.dx + (size_t)t * d.M + m, dz * W[m]);
          atomicAdd(dW + ((size_t)h * d.M + m) * d.E + e, x[m] * dz);
        }
      }
  }
}
