// Normalized gated linear attention in its recurrent form (Eq. 4, Eq. 8), forward and backward, as fp32 CUDA-core
// kernels. One block walks one (batch, query head) along the tokens with the state held in registers. This is the
// exact-arithmetic path: it serves the fp32 mode and every shape the tensor-core path does not take.
//
// Backward (chain rule on Eq. 4/8; v' = [v,1], S' = [S,z], o' = qdot S' = [n,d]):
//   do'_t  = [dO_t/d_t, -(dO_t.o_t)/d_t]         d_t and dO_t.o_t are recomputed in fp32 by the forward sweep (the
//                                                stored o is rounded to the storage type and dqdot cancels heavily)
//   dqdot_t = do'_t S'_t^T                       forward sweep, state rows owned by threads ("row sweep")
//   dS'_t   = sum_{s>=t} decay(t->s) qdot_s^T do'_s   reverse sweeps:
//   dkdot_t = dS'_t v'_t                          rows owned by threads
//   dv'_t   = kdot_t dS'_t                        columns owned by threads
//   dg_s    = sum_{t>=s} (qdot_t*dqdot_t - kdot_t*dkdot_t)   (o' depends on the log-decays only through their running
//             sum), accumulated in the same reverse sweep that produces dkdot.
#include "common.cuh"

namespace lawcat {

constexpr int TB = 8;  // tokens staged in shared memory per step

struct GlaArgs {
  const void *qdot, *kdot, *v, *gate, *o, *dO;
  const float *S0, *z0, *den;
  void *out_o, *d_qdot, *d_kdot, *dgate;
  float *out_den, *S_T, *z_T, *dvh;
  float *bw_qdq;         // [B,T,H,dk] scratch of the backward: qdot*dqdot in fp32 (the gate gradient cancels heavily)
  float *bw_den, *bw_w;  // [B,T,H] scratch of the backward: d_t and the z-column coefficient -(dO_t.n_t)/d_t^2
  int B, T, H, Hkv, dk, dv, gd, gate_mode, normalize;
  float inv_tau, eps;
};

// ------------------------------------------------------------------------------------------------ forward
// Thread (rg, col): column col of S' (col == dv is the z column), rows [rg*R, rg*R+R). o'_t[col] is a sum over rows:
// in-thread over R rows, then over the row groups through shared memory once per staged batch.
template <typename TQ, typename TS, int R>
__global__ void gla_fwd_rec_kernel(GlaArgs a) {
  extern __shared__ __align__(16) float smem[];
  const int dk = a.dk, dv = a.dv, Tn = a.T, H = a.H;
  const int CW = (dv + 1 + 31) / 32 * 32, RG = dk / R;
  float* s_alpha = smem;               // [TB][dk]
  float* s_k = s_alpha + TB * dk;      // [TB][dk]
  float* s_q = s_k + TB * dk;          // [TB][dk]
  float* s_v = s_q + TB * dk;          // [TB][CW]
  float* s_part = s_v + TB * CW;       // [TB][RG][CW]
  const int b = blockIdx.x / H, h = blockIdx.x % H, j = h / (H / a.Hkv);
  const int tid = threadIdx.x, nthr = blockDim.x;
  const int rg = tid / CW, col = tid % CW;
  const bool active = col <= dv;
  const TQ* qdot = (const TQ*)a.qdot;
  const TQ* kdot = (const TQ*)a.kdot;
  const TS* v = (const TS*)a.v;
  const TS* gate = (const TS*)a.gate;
  TS* o = (TS*)a.out_o;
  float S[R];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int row = rg * R + r;
    float s0 = 0.f;
    if (col < dv && a.S0) s0 = a.S0[(((size_t)b * H + h) * dk + row) * dv + col];
    if (col == dv && a.z0) s0 = a.z0[((size_t)b * H + h) * dk + row];
    S[r] = s0;
  }
  for (int t0 = 0; t0 < Tn; t0 += TB) {
    const int nt = min(TB, Tn - t0);
    for (int i = tid; i < nt * dk; i += nthr) {
      const int tok = i / dk, c = i % dk;
      const size_t th = ((size_t)b * Tn + t0 + tok) * H + h;
      s_q[i] = ldf(qdot + th * dk + c);
      s_k[i] = ldf(kdot + th * dk + c);
      s_alpha[i] = expf(log_decay(ldf(gate + th * a.gd + (a.gd == 1 ? 0 : c)), a.gate_mode, a.inv_tau));
    }
    for (int i = tid; i < nt * CW; i += nthr) {
      const int tok = i / CW, e = i % CW;
      s_v[i] = e < dv ? ldf(v + (((size_t)b * Tn + t0 + tok) * a.Hkv + j) * dv + e) : (e == dv ? 1.f : 0.f);
    }
    __syncthreads();
    if (active) {
      for (int tok = 0; tok < nt; ++tok) {
        const float vc = s_v[tok * CW + col];
        const float4* a4 = reinterpret_cast<const float4*>(s_alpha + tok * dk + rg * R);
        const float4* k4 = reinterpret_cast<const float4*>(s_k + tok * dk + rg * R);
        const float4* q4 = reinterpret_cast<const float4*>(s_q + tok * dk + rg * R);
        float acc = 0.f;
#pragma unroll
        for (int r4 = 0; r4 < R / 4; ++r4) {
          const float4 al = a4[r4], kk = k4[r4], qq = q4[r4];
          S[4 * r4 + 0] = fmaf(al.x, S[4 * r4 + 0], kk.x * vc); acc = fmaf(qq.x, S[4 * r4 + 0], acc);
          S[4 * r4 + 1] = fmaf(al.y, S[4 * r4 + 1], kk.y * vc); acc = fmaf(qq.y, S[4 * r4 + 1], acc);
          S[4 * r4 + 2] = fmaf(al.z, S[4 * r4 + 2], kk.z * vc); acc = fmaf(qq.z, S[4 * r4 + 2], acc);
          S[4 * r4 + 3] = fmaf(al.w, S[4 * r4 + 3], kk.w * vc); acc = fmaf(qq.w, S[4 * r4 + 3], acc);
        }
        s_part[(tok * RG + rg) * CW + col] = acc;
      }
    }
    __syncthreads();
    for (int i = tid; i < nt * dv; i += nthr) {
      const int tok = i / dv, e = i % dv;
      float num = 0.f, dn = a.eps;
      for (int g = 0; g < RG; ++g) {
        num += s_part[(tok * RG + g) * CW + e];
        dn += s_part[(tok * RG + g) * CW + dv];
      }
      const size_t th = ((size_t)b * Tn + t0 + tok) * H + h;
      stf(o + th * dv + e, a.normalize ? num / dn : num);
      if (e == 0 && a.out_den) a.out_den[th] = dn;
    }
    __syncthreads();
  }
  if (active) {
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int row = rg * R + r;
      if (col < dv && a.S_T) a.S_T[(((size_t)b * H + h) * dk + row) * dv + col] = S[r];
      if (col == dv && a.z_T) a.z_T[((size_t)b * H + h) * dk + row] = S[r];
    }
  }
}

template <typename TQ, typename TS>
static int gla_fwd_launch(const Ctx& c, GlaArgs& a) {
  const lawcat_params& p = *c.p;
  if (p.B * p.H == 0) return LAWCAT_OK;
  const int RG = p.d_k >= 64 ? 4 : (p.d_k >= 32 ? 2 : 1), R = p.d_k / RG;  // (at most 4 x 160 threads)
  const int CW = (p.d_v + 1 + 31) / 32 * 32;
  const size_t smem = sizeof(float) * ((size_t)3 * TB * p.d_k + (size_t)TB * CW + (size_t)TB * RG * CW);
  const int threads = RG * CW;
  const unsigned grid = p.B * p.H;
  LaunchScope _ls("gla_fwd_rec", c.stream);
  switch (R) {
    case 16: gla_fwd_rec_kernel<TQ, TS, 16><<<grid, threads, smem, c.stream>>>(a); break;
    case 32: gla_fwd_rec_kernel<TQ, TS, 32><<<grid, threads, smem, c.stream>>>(a); break;
    case 64: gla_fwd_rec_kernel<TQ, TS, 64><<<grid, threads, smem, c.stream>>>(a); break;
    default: return LAWCAT_ERR_UNSUPPORTED;
  }
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

static GlaArgs base_args(const lawcat_params& p) {
  GlaArgs a{};
  a.B = p.B; a.T = p.T; a.H = p.H; a.Hkv = p.H_kv; a.dk = p.d_k; a.dv = p.d_v; a.gd = p.gate_dim;
  a.gate_mode = p.gate_mode; a.normalize = p.normalize; a.inv_tau = 1.f / p.gate_tau; a.eps = p.eps;
  return a;
}

int launch_gla_fwd_rec(const Ctx& c, const void* qdot, const void* kdot, bool qk_f32, const void* v,
                       const void* gate, const float* S0, const float* z0, void* o, float* den, float* S_T,
                       float* z_T) {
  const lawcat_params& p = *c.p;
  GlaArgs a = base_args(p);
  a.qdot = qdot; a.kdot = kdot; a.v = v; a.gate = gate; a.S0 = S0; a.z0 = z0;
  a.out_o = o; a.out_den = den; a.S_T = S_T; a.z_T = z_T;
  if (p.T == 0) {  // empty sequence: the state passes through unchanged
    const size_t nS = sizeof(float) * (size_t)p.B * p.H * p.d_k * p.d_v, nz = sizeof(float) * (size_t)p.B * p.H * p.d_k;
    if (S_T && (S0 ? cudaMemcpyAsync(S_T, S0, nS, cudaMemcpyDeviceToDevice, c.stream) : cudaMemsetAsync(S_T, 0, nS, c.stream)))
      return LAWCAT_ERR_CUDA;
    if (z_T && (z0 ? cudaMemcpyAsync(z_T, z0, nz, cudaMemcpyDeviceToDevice, c.stream) : cudaMemsetAsync(z_T, 0, nz, c.stream)))
      return LAWCAT_ERR_CUDA;
    return LAWCAT_OK;
  }
  if (p.dtype == LAWCAT_F32) return gla_fwd_launch<float, float>(c, a);
  if (qk_f32) return gla_fwd_launch<float, bf16>(c, a);
  return gla_fwd_launch<bf16, bf16>(c, a);
}

// ------------------------------------------------------------------------------------------------ backward sweeps
// Stage do'_t for a batch of tokens from dO and the two per-token scalars the forward sweep left in scratch.
template <typename TS>
__device__ __forceinline__ void stage_dop(const GlaArgs& a, float* s_dop, int b, int h, int t0, int nt, int tid,
                                          int nthr) {
  const int dv = a.dv;
  const TS* dO = (const TS*)a.dO;
  for (int i = tid; i < nt * (dv + 1); i += nthr) {
    const int tok = i / (dv + 1), e = i % (dv + 1);
    const size_t th = ((size_t)b * a.T + t0 + tok) * a.H + h;
    float val;
    if (e < dv) val = ldf(dO + th * dv + e) * (a.normalize ? 1.f / a.bw_den[th] : 1.f);
    else val = a.normalize ? a.bw_w[th] : 0.f;
    s_dop[i] = val;
  }
}

// Row sweeps. Thread (c, seg): row c of S' (or dS'), columns [seg*CS, seg*CS+CS); seg 0 also owns the z column.
// MODE 0: forward in time, recompute S'_t, emit dqdot_t.  MODE 1: backward in time, carry dS', emit dkdot_t and dgate_t.
template <typename TS, int CS, int MODE>
__global__ void gla_bwd_row_kernel(GlaArgs a) {
  extern __shared__ __align__(16) float smem[];
  const int dk = a.dk, dv = a.dv, Tn = a.T, H = a.H, NSEG = dv / CS;
  float* s_alpha = smem;                 // [TB][dk]
  float* s_k = s_alpha + TB * dk;        // [TB][dk]
  float* s_q = s_k + TB * dk;            // [TB][dk]   (MODE 1)
  float* s_dq = s_q + TB * dk;           // [TB][dk]   MODE 0: output dqdot ; MODE 1: input dqdot
  float* s_out = s_dq + TB * dk;         // [TB][dk]   MODE 1: dkdot
  float* s_dg = s_out + TB * dk;         // [TB][dk]   MODE 1: running dg
  float* s_v = s_dg + TB * dk;           // [TB][dv]
  float* s_dop = s_v + TB * dv;          // [TB][dv+1]
  const int b = blockIdx.x / H, h = blockIdx.x % H, j = h / (H / a.Hkv);
  const int tid = threadIdx.x, nthr = blockDim.x;
  const int c = min(tid / NSEG, dk - 1), seg = tid % NSEG;
  const bool rowact = tid < dk * NSEG;  // the block is padded to whole warps
  const TS* qdot = (const TS*)a.qdot;
  const TS* kdot = (const TS*)a.kdot;
  const TS* v = (const TS*)a.v;
  const TS* gate = (const TS*)a.gate;
  float S[CS], z = 0.f, accg = 0.f;
#pragma unroll
  for (int e = 0; e < CS; ++e)
    S[e] = (MODE == 0 && a.S0) ? a.S0[(((size_t)b * H + h) * dk + c) * dv + seg * CS + e] : 0.f;
  if (MODE == 0 && a.z0) z = a.z0[((size_t)b * H + h) * dk + c];
  const int nbatch = (Tn + TB - 1) / TB;
  for (int bi = 0; bi < nbatch; ++bi) {
    const int t0 = (MODE == 0 ? bi : nbatch - 1 - bi) * TB;
    const int nt = min(TB, Tn - t0);
    for (int i = tid; i < nt * dk; i += nthr) {
      const int tok = i / dk, cc = i % dk;
      const size_t th = ((size_t)b * Tn + t0 + tok) * H + h;
      s_k[i] = ldf(kdot + th * dk + cc);
      s_alpha[i] = expf(log_decay(ldf(gate + th * a.gd + (a.gd == 1 ? 0 : cc)), a.gate_mode, a.inv_tau));
      s_q[i] = ldf(qdot + th * dk + cc);
      if (MODE == 1) s_dq[i] = a.bw_qdq[th * dk + cc];
    }
    for (int i = tid; i < nt * dv; i += nthr) {
      const int tok = i / dv, e = i % dv;
      s_v[i] = ldf(v + (((size_t)b * Tn + t0 + tok) * a.Hkv + j) * dv + e);
    }
    if (MODE == 0) {
      for (int i = tid; i < nt * dv; i += nthr) {  // raw dO; the scaling by 1/d_t follows once d_t is known
        const int tok = i / dv, e = i % dv;
        s_dop[tok * (dv + 1) + e] = ldf((const TS*)a.dO + (((size_t)b * Tn + t0 + tok) * H + h) * dv + e);
      }
    } else {
      stage_dop<TS>(a, s_dop, b, h, t0, nt, tid, nthr);
    }
    __syncthreads();
    if (MODE == 0) {
      // A_c = sum_e dO_e S'_t[c][e] and z_t[c] per row; then d_t = qdot.z + eps, dO.n = qdot.A (sums over rows) and
      // dqdot_c = A_c/d_t - (dO.n) z_c/d_t^2
      for (int tok = 0; tok < nt; ++tok) {
        const float al = s_alpha[tok * dk + c], kk = s_k[tok * dk + c];
        const float* vv = s_v + tok * dv + seg * CS;
        const float* dp = s_dop + tok * (dv + 1) + seg * CS;
        float A = 0.f;
#pragma unroll
        for (int e = 0; e < CS; ++e) {
          S[e] = fmaf(al, S[e], kk * vv[e]);
          A = fmaf(dp[e], S[e], A);
        }
        if (seg == 0) z = fmaf(al, z, kk);
        for (int o = NSEG >> 1; o > 0; o >>= 1) A += __shfl_xor_sync(0xffffffffu, A, o);
        if (seg == 0 && rowact) {
          s_dq[tok * dk + c] = A;
          s_out[tok * dk + c] = z;
        }
      }
      __syncthreads();
      {
        const int warp = tid >> 5, lane = tid & 31, nwarp = nthr >> 5;
        for (int tok = warp; tok < nt; tok += nwarp) {
          float dn = 0.f, dOn = 0.f;
          for (int cc = lane; cc < dk; cc += 32) {
            dn = fmaf(s_q[tok * dk + cc], s_out[tok * dk + cc], dn);
            dOn = fmaf(s_q[tok * dk + cc], s_dq[tok * dk + cc], dOn);
          }
          dn = warp_sum(dn) + a.eps;
          dOn = warp_sum(dOn);
          if (lane == 0) {
            const size_t th = ((size_t)b * Tn + t0 + tok) * H + h;
            s_dg[2 * tok] = 1.f / dn;
            s_dg[2 * tok + 1] = -dOn / (dn * dn);
            a.bw_den[th] = dn;
            a.bw_w[th] = -dOn / (dn * dn);
          }
        }
      }
    } else {
      for (int tok = nt - 1; tok >= 0; --tok) {
        const float al = s_alpha[tok * dk + c], kk = s_k[tok * dk + c], qq = s_q[tok * dk + c];
        const float* vv = s_v + tok * dv + seg * CS;
        const float* dp = s_dop + tok * (dv + 1) + seg * CS;
        float dkk = 0.f;
#pragma unroll
        for (int e = 0; e < CS; ++e) {
          S[e] = fmaf(qq, dp[e], S[e]);
          dkk = fmaf(S[e], vv[e], dkk);
        }
        if (seg == 0) {
          z = fmaf(qq, s_dop[tok * (dv + 1) + dv], z);
          dkk += z;
        }
        for (int o = NSEG >> 1; o > 0; o >>= 1) dkk += __shfl_xor_sync(0xffffffffu, dkk, o);
#pragma unroll
        for (int e = 0; e < CS; ++e) S[e] *= al;
        z *= al;
        if (seg == 0 && rowact) {
          accg += s_dq[tok * dk + c] - kk * dkk;
          s_out[tok * dk + c] = dkk;
          s_dg[tok * dk + c] = accg;
        }
      }
    }
    __syncthreads();
    if (MODE == 0) {
      for (int i = tid; i < nt * dk; i += nthr) {
        const int tok = i / dk;
        const size_t th = ((size_t)b * Tn + t0 + tok) * H + h;
        const float dq = a.normalize ? fmaf(s_dq[i], s_dg[2 * tok], s_out[i] * s_dg[2 * tok + 1]) : s_dq[i];
        stf((TS*)a.d_qdot + th * dk + i % dk, dq);
        a.bw_qdq[th * dk + i % dk] = s_q[i] * dq;
      }
    } else {
      for (int i = tid; i < nt * dk; i += nthr) {
        const int tok = i / dk, cc = i % dk;
        const size_t th = ((size_t)b * Tn + t0 + tok) * H + h;
        stf((TS*)a.d_kdot + th * dk + cc, s_out[i]);
        if (a.gd != 1) {
          const float araw = ldf(gate + th * a.gd + cc);
          stf((TS*)a.dgate + th * a.gd + cc, s_dg[i] * log_decay_grad(araw, a.gate_mode, a.inv_tau));
        }
      }
      if (a.gd == 1) {
        const int warp = tid >> 5, lane = tid & 31, nwarp = (nthr + 31) >> 5;
        for (int tok = warp; tok < nt; tok += nwarp) {
          float s = 0.f;
          for (int cc = lane; cc < dk; cc += 32) s += s_dg[tok * dk + cc];
          s = warp_sum(s);
          if (lane == 0) {
            const size_t th = ((size_t)b * Tn + t0 + tok) * H + h;
            stf((TS*)a.dgate + th, s * log_decay_grad(ldf(gate + th), a.gate_mode, a.inv_tau));
          }
        }
      }
    }
    __syncthreads();
  }
}

// Column sweep, backward in time: thread (rg, col) owns column col < dv of dS', rows [rg*R, rg*R+R); emits
// dv'_t[col] = sum_rows kdot_t[row] dS'_t[row][col] per query head into an fp32 scratch [B,T,H,dv].
template <typename TS, int R>
__global__ void gla_bwd_col_kernel(GlaArgs a) {
  extern __shared__ __align__(16) float smem[];
  const int dk = a.dk, dv = a.dv, Tn = a.T, H = a.H, RG = dk / R;
  float* s_alpha = smem;               // [TB][dk]
  float* s_k = s_alpha + TB * dk;      // [TB][dk]
  float* s_q = s_k + TB * dk;          // [TB][dk]
  float* s_dop = s_q + TB * dk;        // [TB][dv+1]
  float* s_part = s_dop + TB * (dv + 1);  // [TB][RG][dv]
  const int b = blockIdx.x / H, h = blockIdx.x % H;
  const int tid = threadIdx.x, nthr = blockDim.x;
  const int rg = min(tid / dv, RG - 1), col = tid % dv;
  const bool colact = tid < RG * dv;  // the block is padded to whole warps
  const TS* qdot = (const TS*)a.qdot;
  const TS* kdot = (const TS*)a.kdot;
  const TS* gate = (const TS*)a.gate;
  float dS[R];
#pragma unroll
  for (int r = 0; r < R; ++r) dS[r] = 0.f;
  const int nbatch = (Tn + TB - 1) / TB;
  for (int bi = nbatch - 1; bi >= 0; --bi) {
    const int t0 = bi * TB, nt = min(TB, Tn - t0);
    for (int i = tid; i < nt * dk; i += nthr) {
      const int tok = i / dk, cc = i % dk;
      const size_t th = ((size_t)b * Tn + t0 + tok) * H + h;
      s_q[i] = ldf(qdot + th * dk + cc);
      s_k[i] = ldf(kdot + th * dk + cc);
      s_alpha[i] = expf(log_decay(ldf(gate + th * a.gd + (a.gd == 1 ? 0 : cc)), a.gate_mode, a.inv_tau));
    }
    stage_dop<TS>(a, s_dop, b, h, t0, nt, tid, nthr);
    __syncthreads();
    for (int tok = nt - 1; tok >= 0; --tok) {
      const float dc = s_dop[tok * (dv + 1) + col];
      const float4* a4 = reinterpret_cast<const float4*>(s_alpha + tok * dk + rg * R);
      const float4* k4 = reinterpret_cast<const float4*>(s_k + tok * dk + rg * R);
      const float4* q4 = reinterpret_cast<const float4*>(s_q + tok * dk + rg * R);
      float acc = 0.f;
#pragma unroll
      for (int r4 = 0; r4 < R / 4; ++r4) {
        const float4 al = a4[r4], kk = k4[r4], qq = q4[r4];
        dS[4 * r4 + 0] = fmaf(qq.x, dc, dS[4 * r4 + 0]); acc = fmaf(kk.x, dS[4 * r4 + 0], acc); dS[4 * r4 + 0] *= al.x;
        dS[4 * r4 + 1] = fmaf(qq.y, dc, dS[4 * r4 + 1]); acc = fmaf(kk.y, dS[4 * r4 + 1], acc); dS[4 * r4 + 1] *= al.y;
        dS[4 * r4 + 2] = fmaf(qq.z, dc, dS[4 * r4 + 2]); acc = fmaf(kk.z, dS[4 * r4 + 2], acc); dS[4 * r4 + 2] *= al.z;
        dS[4 * r4 + 3] = fmaf(qq.w, dc, dS[4 * r4 + 3]); acc = fmaf(kk.w, dS[4 * r4 + 3], acc); dS[4 * r4 + 3] *= al.w;
      }
      if (colact) s_part[(tok * RG + rg) * dv + col] = acc;
    }
    __syncthreads();
    for (int i = tid; i < nt * dv; i += nthr) {
      const int tok = i / dv, e = i % dv;
      float s = 0.f;
      for (int g = 0; g < RG; ++g) s += s_part[(tok * RG + g) * dv + e];
      a.dvh[(((size_t)b * Tn + t0 + tok) * H + h) * dv + e] = s;
    }
    __syncthreads();
  }
}

// dv[b,t,j,:] = sum over the G query heads of group j of the per-head scratch (keys and values are shared in a group)
template <typename TS>
__global__ void dv_group_reduce_kernel(const float* __restrict__ dvh, TS* __restrict__ dv_out, size_t total, int Hkv,
                                       int G, int dv) {
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int e = (int)(idx % dv);
  const size_t bt_j = idx / dv;
  const int j = (int)(bt_j % Hkv);
  const size_t bt = bt_j / Hkv;
  float s = 0.f;
  for (int g = 0; g < G; ++g) s += dvh[((bt * Hkv + j) * G + g) * dv + e];
  stf(dv_out + idx, s);
}

template <typename TS>
static int gla_bwd_typed(const Ctx& c, GlaArgs& a, void* dv_out) {
  const lawcat_params& p = *c.p;
  const int dk = p.d_k, dv = p.d_v;
  const unsigned grid = p.B * p.H;
  const int CS = 16, NSEG = dv / CS;  // 16 state columns per thread: more, shorter dependent chains per token
  const size_t smem_row = sizeof(float) * ((size_t)6 * TB * dk + (size_t)TB * dv + (size_t)TB * (dv + 1));
  const int RG = dk >= 64 ? 4 : (dk >= 32 ? 2 : 1), R = dk / RG;
  const size_t smem_col = sizeof(float) * ((size_t)3 * TB * dk + (size_t)TB * (dv + 1) + (size_t)TB * RG * dv);
  const int row_thr = (dk * NSEG + 31) / 32 * 32, col_thr = (RG * dv + 31) / 32 * 32;
  // sweep 1: dqdot (forward in time) ; sweep 2: per-head dv (backward in time) ; sweep 3: dkdot + dgate
  LAWCAT_LAUNCH("gla_bwd_row_fwd", c.stream,
                gla_bwd_row_kernel<TS, 16, 0><<<grid, row_thr, smem_row, c.stream>>>(a));
  LAWCAT_CHECK_LAUNCH();
  if (R != 16 && R != 32 && R != 64) return LAWCAT_ERR_UNSUPPORTED;
  LAWCAT_LAUNCH("gla_bwd_col", c.stream,
                if (R == 16) gla_bwd_col_kernel<TS, 16><<<grid, col_thr, smem_col, c.stream>>>(a);
                else if (R == 32) gla_bwd_col_kernel<TS, 32><<<grid, col_thr, smem_col, c.stream>>>(a);
                else gla_bwd_col_kernel<TS, 64><<<grid, col_thr, smem_col, c.stream>>>(a));
  LAWCAT_CHECK_LAUNCH();
  LAWCAT_LAUNCH("gla_bwd_row_rev", c.stream,
                gla_bwd_row_kernel<TS, 16, 1><<<grid, row_thr, smem_row, c.stream>>>(a));
  LAWCAT_CHECK_LAUNCH();
  const size_t total = (size_t)p.B * p.T * p.H_kv * dv;
  LAWCAT_LAUNCH("dv_group_reduce", c.stream,
                dv_group_reduce_kernel<TS><<<(unsigned)((total + 255) / 256), 256, 0, c.stream>>>(
                    a.dvh, (TS*)dv_out, total, p.H_kv, p.H / p.H_kv, dv));
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

int launch_gla_bwd_rec(const Ctx& c, const void* qdot, const void* kdot, const void* v, const void* gate,
                       const float* S0, const float* z0, const void* o, const float* den, const void* dO,
                       void* d_qdot, void* d_kdot, void* dv, void* dgate, void* ws) {
  const lawcat_params& p = *c.p;
  if ((size_t)p.B * p.T * p.H == 0) return LAWCAT_OK;
  GlaArgs a = base_args(p);
  a.qdot = qdot; a.kdot = kdot; a.v = v; a.gate = gate; a.S0 = S0; a.z0 = z0; a.o = o; a.den = den; a.dO = dO;
  a.d_qdot = d_qdot; a.d_kdot = d_kdot; a.dgate = dgate; a.dvh = (float*)ws;
  const size_t n_dvh = align_up(sizeof(float) * (size_t)p.B * p.T * p.H * p.d_v, 256);
  const size_t n_bth = align_up(sizeof(float) * (size_t)p.B * p.T * p.H, 256);
  a.bw_den = (float*)((char*)ws + n_dvh);
  a.bw_w = (float*)((char*)ws + n_dvh + n_bth);
  a.bw_qdq = (float*)((char*)ws + n_dvh + 2 * n_bth);
  (void)o; (void)den;
  if (p.dtype == LAWCAT_F32) return gla_bwd_typed<float>(c, a, dv);
  return gla_bwd_typed<bf16>(c, a, dv);
}

}  // namespace lawcat
