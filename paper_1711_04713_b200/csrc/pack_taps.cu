// LPConvolution with very few input channels (paper Sec. 2; the first layer of an image network:
// 3 channels, 3x3 taps) as a packed GEMM.
//
// With C <= 4 channels the implicit-GEMM path would move one mostly empty 32-byte K-block per tap
// (9 blocks of which 27 bytes in 288 are real for an RGB 3x3 layer).  Instead the R*S*C <= 32
// real reduction elements of every output pixel are gathered once into one 32-byte row
//   P[m][t*C + c] = x[n, oh*stride + r - pad, ow*stride + s - pad, c],   t = r*S + s
// (zero outside the image, zero beyond R*S*C), per byte plane, the weights likewise into
// W'[k][t*C + c], and the layer runs as the inner product P * W'^T on the tensor-core path
// with its usual fused epilogue.  The packed planes live in the caller's workspace.
#include "common.cuh"

namespace adaption {

int num_sms();

namespace {

constexpr int kPackK = 32;   // bytes per packed row (one 32-byte K-block)

struct PackParams {
  const uint8_t* src[2];     // byte planes of the source tensor (second may be null)
  uint8_t* dst[2];           // packed planes, rows of kPackK bytes
  long long rows;            // output pixels (activations) or output channels (weights)
  long long c_stride;        // source channel pitch
  int planes;
  int is_weight;             // source is [rows][R*S][c_stride]: no geometry, always in bounds
  int H, W, OH, OW, R, S, pad_h, pad_w, stride_h, stride_w;
};

// One thread gathers the packed rows of one output pixel (or weight row) in every plane, so that
// the index arithmetic is done once.  C is a template parameter so that every byte position
// t*C + c is known at compile time and the eight output words stay in registers.  Each tap is read
// as one aligned 32-bit word (the channel pitch is a multiple of 16 bytes and C <= 4), of which the
// low C bytes are used.  Pixels whose whole window lies inside the image skip the bounds tests.
template <int C, bool CHECKED>
__device__ __forceinline__ void pack_row(const uint8_t* __restrict__ src, long long base, long long tap_pitch,
                                         long long row_pitch, int taps, int S, int ih0, int iw0, int H, int W,
                                         uint8_t* __restrict__ dst) {
  constexpr int kMaxTaps = kPackK / C;
  uint32_t out[kPackK / 4];
#pragma unroll
  for (int j = 0; j < kPackK / 4; ++j) out[j] = 0u;
  int r = 0, s = 0;
  long long off = base;                 // element offset of the current tap
#pragma unroll
  for (int t = 0; t < kMaxTaps; ++t) {
    uint32_t v = 0u;
    if (t < taps) {
      bool inside = true;
      if (CHECKED) {
        const int ih = ih0 + r, iw = iw0 + s;
        inside = ih >= 0 && ih < H && iw >= 0 && iw < W;
      }
      if (inside) v = __ldg(reinterpret_cast<const unsigned int*>(src + off));
    }
    v &= 0xffffffffu >> (32 - 8 * C);
    // bytes t*C .. t*C + C - 1 of the packed row (may straddle two words)
    const int k0 = t * C;
    const int w0 = k0 >> 2, sh = (k0 & 3) * 8;
    out[w0] |= v << sh;
    if (sh + 8 * C > 32) out[w0 + 1] |= v >> (32 - sh);
    off += tap_pitch;
    if (++s == S) { s = 0; ++r; off += row_pitch - (long long)S * tap_pitch; }
  }
  uint4* d = reinterpret_cast<uint4*>(dst);
  d[0] = make_uint4(out[0], out[1], out[2], out[3]);
  d[1] = make_uint4(out[4], out[5], out[6], out[7]);
}

template <int C>
__global__ void __launch_bounds__(256) pack_taps_kernel(const PackParams p) {
  pdl_prologue();
  const int taps = p.R * p.S;
  for (long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x; m < p.rows;
       m += (long long)gridDim.x * blockDim.x) {
    if (p.is_weight) {
      // [rows][R*S][c_stride]: consecutive taps are one pitch apart, always in bounds
      for (int plane = 0; plane < p.planes; ++plane)
        pack_row<C, false>(p.src[plane], m * (long long)taps * p.c_stride, p.c_stride, (long long)p.S * p.c_stride,
                           taps, p.S, 0, 0, 0, 0, p.dst[plane] + m * kPackK);
      continue;
    }
    // pixel index -> (image, row, column); 32-bit arithmetic whenever the index fits
    int ow, oh;
    long long img;
    if (p.rows <= 0x7fffffffll) {
      const unsigned mu = (unsigned)m, rest = mu / (unsigned)p.OW;
      ow = (int)(mu - rest * (unsigned)p.OW);
      const unsigned im = rest / (unsigned)p.OH;
      oh = (int)(rest - im * (unsigned)p.OH);
      img = im;
    } else {
      ow = (int)(m % p.OW);
      const long long rest = m / p.OW;
      oh = (int)(rest % p.OH);
      img = rest / p.OH;
    }
    const int ih0 = oh * p.stride_h - p.pad_h, iw0 = ow * p.stride_w - p.pad_w;
    const long long base = ((img * p.H + ih0) * (long long)p.W + iw0) * p.c_stride;
    const long long row_pitch = (long long)p.W * p.c_stride;
    const bool interior = ih0 >= 0 && ih0 + p.R <= p.H && iw0 >= 0 && iw0 + p.S <= p.W;
    for (int plane = 0; plane < p.planes; ++plane) {
      if (interior)
        pack_row<C, false>(p.src[plane], base, p.c_stride, row_pitch, taps, p.S, ih0, iw0, p.H, p.W,
                           p.dst[plane] + m * kPackK);
      else
        pack_row<C, true>(p.src[plane], base, p.c_stride, row_pitch, taps, p.S, ih0, iw0, p.H, p.W,
                          p.dst[plane] + m * kPackK);
    }
  }
}

int launch_pack(const PackParams& p, int C, cudaStream_t stream) {
  const long long total = p.rows;
  if (total == 0) return ADAPTION_OK;
  long long blocks = (total + 255) / 256;
  const long long cap = (long long)num_sms() * 16;
  if (blocks > cap) blocks = cap;
  switch (C) {
    case 1: launch_after_predecessor(pack_taps_kernel<1>, dim3((unsigned)blocks), dim3(256), stream, p); break;
    case 2: launch_after_predecessor(pack_taps_kernel<2>, dim3((unsigned)blocks), dim3(256), stream, p); break;
    case 3: launch_after_predecessor(pack_taps_kernel<3>, dim3((unsigned)blocks), dim3(256), stream, p); break;
    default: launch_after_predecessor(pack_taps_kernel<4>, dim3((unsigned)blocks), dim3(256), stream, p); break;
  }
  return cuda_status(cudaGetLastError(), "pack_taps_kernel launch");
}

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

struct PackLayout {
  size_t a_plane, w_plane;     // bytes of one packed activation / weight plane
  size_t total;
};

PackLayout layout_of(const GemmProblem& g) {
  PackLayout l;
  l.a_plane = align256((size_t)g.M * kPackK);
  l.w_plane = align256((size_t)g.N * kPackK);
  l.total = 2 * l.a_plane + 2 * l.w_plane;
  return l;
}

// the inner product that the packed layer becomes
GemmProblem packed_problem(const GemmProblem& g, uint8_t* ws) {
  const PackLayout l = layout_of(g);
  GemmProblem q = g;
  q.is_conv = false;
  q.K = kPackK;
  const bool x2 = g.x.fmt.n_bits > 8, w2 = g.w.fmt.n_bits > 8;
  q.x.lo = ws;
  q.x.hi = x2 ? ws + l.a_plane : nullptr;
  q.x.q16 = nullptr;
  q.x.c_stride = kPackK;
  q.w.lo = ws + 2 * l.a_plane;
  q.w.hi = w2 ? ws + 2 * l.a_plane + l.w_plane : nullptr;
  q.w.q16 = nullptr;
  q.w.c_stride = kPackK;
  q.workspace = nullptr;
  q.workspace_bytes = 0;
  return q;
}

}  // namespace

// Few channels, all taps of a pixel fit one 32-byte row, enough rows to be worth a tensor-core
// launch, and the packed inner product is one the tensor-core path takes without scratch memory.
bool pack_taps_applicable(const GemmProblem& g) {
  if (!g.is_conv || g.cs.C > 4 || (int64_t)g.cs.R * g.cs.S * g.cs.C > kPackK) return false;
  if (g.M < 1024 || g.x.c_stride % 16 != 0 || g.x.c_stride != g.w.c_stride) return false;
  uint8_t* fake = reinterpret_cast<uint8_t*>(uintptr_t(256));
  const GemmProblem q = packed_problem(g, fake);
  return tensor_path_supported(q) && tensor_path_workspace(q) == 0;
}

size_t pack_taps_workspace(const GemmProblem& g) { return layout_of(g).total; }

// whether the packed inner product can store horizontal pair maxima (GemmProblem::pool_w)
bool pack_taps_can_pool(const GemmProblem& g) {
  uint8_t* fake = reinterpret_cast<uint8_t*>(uintptr_t(256));
  return (g.OW & 1) == 0 && tensor_path_can_pool(packed_problem(g, fake));
}

int launch_pack_taps(const GemmProblem& g) {
  uint8_t* ws = static_cast<uint8_t*>(g.workspace);
  const GemmProblem q = packed_problem(g, ws);
  PackParams p{};
  p.c_stride = g.x.c_stride;
  p.H = g.cs.H; p.W = g.cs.W; p.OH = g.OH; p.OW = g.OW; p.R = g.cs.R; p.S = g.cs.S;
  p.pad_h = g.cs.pad_h; p.pad_w = g.cs.pad_w; p.stride_h = g.cs.stride_h; p.stride_w = g.cs.stride_w;
  // activations
  p.is_weight = 0;
  p.rows = g.M;
  p.planes = q.x.hi != nullptr ? 2 : 1;
  p.src[0] = static_cast<const uint8_t*>(g.x.lo); p.dst[0] = static_cast<uint8_t*>(q.x.lo);
  p.src[1] = static_cast<const uint8_t*>(g.x.hi); p.dst[1] = static_cast<uint8_t*>(q.x.hi);
  int rc = launch_pack(p, g.cs.C, g.stream);
  if (rc != ADAPTION_OK) return rc;
  // weights
  p.is_weight = 1;
  p.rows = g.N;
  p.planes = q.w.hi != nullptr ? 2 : 1;
  p.src[0] = static_cast<const uint8_t*>(g.w.lo); p.dst[0] = static_cast<uint8_t*>(q.w.lo);
  p.src[1] = static_cast<const uint8_t*>(g.w.hi); p.dst[1] = static_cast<uint8_t*>(q.w.hi);
  rc = launch_pack(p, g.cs.C, g.stream);
  if (rc != ADAPTION_OK) return rc;
  return launch_tensor(q);
}

}  // namespace adaption
