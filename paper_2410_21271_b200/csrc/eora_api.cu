// C ABI of libeora_linear (declared in include/eora_linear.h): argument checking, memory
// ownership and dispatch.  All arithmetic of the layer lives in the kernels of the other files.
#include <new>
#include "eora_common.cuh"

using namespace eora;

struct eora_linear {
  Handle h;
};

namespace {

inline int64_t align_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct Carve {
  char* base;
  int64_t off;
  template <typename T>
  T* take(int64_t bytes) {
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += align_up(bytes, 256);
    return p;
  }
};

void wmat_shape(WMat& m, int fmt, int rows, int k_red, int group) {
  m.fmt = fmt;
  m.n_rows = (int)align_up(rows, 16);
  m.k_red = (int)align_up(k_red, 128);
  m.group = group > 0 ? group : m.k_red;
  if (m.group > m.k_red) m.group = m.k_red;
  m.nt = m.n_rows / 16;
  m.kc = m.k_red / 64;
  m.np = m.k_red / 128;
  m.sz2 = (m.group % 128) ? 1 : 0;
  m.blob = blob_bytes(fmt, m.sz2);
  m.q = nullptr;
}

void wmat_carve(WMat& m, Carve& c) {
  if (m.fmt == FMT_NONE) return;
  m.q = c.take<uint8_t>(wmat_q_bytes(m));
}

int check_config(const eora_linear_config& c) {
  if (c.d_in <= 0 || c.d_out <= 0 || c.rank < 0 || c.max_m < 1) return EORA_ERR_BAD_SHAPE;
  if (c.d_in % 128 || c.d_out % 32 || c.rank % 8) return EORA_ERR_BAD_SHAPE;
  if (c.w_format == EORA_W_QUANT) {
    if (c.w_bits != 3 && c.w_bits != 4) return EORA_ERR_UNSUPPORTED;
    if (c.w_group <= 0 || c.w_group % 64 || c.d_in % c.w_group) return EORA_ERR_BAD_SHAPE;
  } else if (c.w_format == EORA_W_SPARSE24_Q4) {
    if (c.w_bits != 4) return EORA_ERR_UNSUPPORTED;
    if (c.w_group <= 0 || c.w_group % 64 || c.d_in % c.w_group) return EORA_ERR_BAD_SHAPE;
  } else if (c.w_format != EORA_W_SPARSE24) {
    return EORA_ERR_UNSUPPORTED;
  }
  if (c.ab_format != EORA_AB_F16 && c.ab_format != EORA_AB_Q4 && c.ab_format != EORA_AB_Q8 && c.ab_format != EORA_AB_Q3)
    return EORA_ERR_UNSUPPORTED;
  if (c.rank > 0 && (c.ab_format == EORA_AB_Q4 || c.ab_format == EORA_AB_Q3)) {
    if (c.rank % 64 || c.ab_group <= 0 || c.ab_group % 64 || c.d_in % c.ab_group) return EORA_ERR_BAD_SHAPE;
    int gb = c.ab_group < c.rank ? c.ab_group : c.rank;
    if (c.rank % gb) return EORA_ERR_BAD_SHAPE;
  }
  if (c.x_dtype != EORA_X_F16 && c.x_dtype != EORA_X_BF16) return EORA_ERR_UNSUPPORTED;
  if (c.y_dtype != EORA_Y_F16 && c.y_dtype != EORA_Y_BF16 && c.y_dtype != EORA_Y_F32) return EORA_ERR_UNSUPPORTED;
  if (c.kernel_policy != EORA_POLICY_AUTO && c.kernel_policy != EORA_POLICY_GENERIC && c.kernel_policy != EORA_POLICY_TMEM_DECODE)
    return EORA_ERR_UNSUPPORTED;
  return EORA_OK;
}

int y_elem_bytes(int y_dtype) { return y_dtype == EORA_Y_F32 ? 4 : 2; }

int pick_path(const Handle* h, int m) {
  if (h->cfg.kernel_policy == EORA_POLICY_GENERIC) return EORA_PATH_GENERIC;
  // The decode family streams the weights once per eight tokens.  From two passes on (m > 8) one launch of the
  // tensor-core family is cheaper: for up to 64 tokens it splits the reduction axis over several CTAs per tile, so it
  // is no longer a chain over all of d_in (measured, 4-bit q-shaped layer, 16 tokens: 23.6 us in two passes, 17 us so).
  if (decode_tc_supported(h, m)) return EORA_PATH_DECODE;   // EORA_POLICY_TMEM_DECODE: one pass over the weights per sixteen tokens
  const bool dec = m <= 64 && decode_supported(h, m), pre = prefill_supported(h, m);
  if (dec && pre) return EORA_PATH_PREFILL;
  if (dec) return EORA_PATH_DECODE;
  if (pre) return EORA_PATH_PREFILL;
  return EORA_PATH_GENERIC;
}

}  // namespace

extern "C" {

int eora_version(void) { return 100; }

const char* eora_status_string(int s) {
  switch (s) {
    case EORA_OK: return "ok";
    case EORA_ERR_NULL_ARG: return "null argument";
    case EORA_ERR_BAD_SHAPE: return "bad shape";
    case EORA_ERR_UNSUPPORTED: return "unsupported format or option";
    case EORA_ERR_MISALIGNED: return "pointer not 16-byte aligned";
    case EORA_ERR_M_TOO_LARGE: return "m exceeds max_m";
    case EORA_ERR_CUDA: return "CUDA runtime error";
    case EORA_ERR_DEVICE_TIMEOUT: return "bounded device-side wait ran out";
    default: return "unknown status";
  }
}

}  // extern "C"

namespace {

int check_weights(const eora_linear_config& c, const eora_linear_weights& w) {
  const bool scaled_w = c.w_format != EORA_W_SPARSE24, meta_w = c.w_format == EORA_W_SPARSE24_Q4;
  if (!w.w_codes || !w.w_zeros || (scaled_w && !w.w_scales) || (meta_w && !w.w_meta)) return EORA_ERR_NULL_ARG;
  if (!aligned16(w.w_codes) || !aligned16(w.w_zeros) || !aligned16(w.w_scales) || (meta_w && !aligned16(w.w_meta)))
    return EORA_ERR_MISALIGNED;
  if (c.rank > 0) {
    if (!w.a || !w.b) return EORA_ERR_NULL_ARG;
    if (!aligned16(w.a) || !aligned16(w.b)) return EORA_ERR_MISALIGNED;
    if (c.ab_format != EORA_AB_F16) {
      if (!w.a_scales || !w.a_zeros || !w.b_scales || !w.b_zeros) return EORA_ERR_NULL_ARG;
      if (!aligned16(w.a_scales) || !aligned16(w.a_zeros) || !aligned16(w.b_scales) || !aligned16(w.b_zeros))
        return EORA_ERR_MISALIGNED;
    }
  }
  return EORA_OK;
}

// Internal format and group of the backbone.
int backbone_fmt(const eora_linear_config& c) {
  if (c.w_format == EORA_W_SPARSE24) return FMT_SP24;
  if (c.w_format == EORA_W_SPARSE24_Q4) return FMT_SQ4;
  return c.w_bits == 4 ? FMT_Q4 : FMT_Q3;
}
int backbone_group(const eora_linear_config& c) { return c.w_format == EORA_W_SPARSE24 ? 0 : c.w_group; }

cudaError_t repack_backbone(const WMat& dst, const eora_linear_config& c, const eora_linear_weights& w, int d_out, cudaStream_t s,
                            int nt_sub) {
  if (c.w_format == EORA_W_QUANT) return launch_repack_quant(dst, w.w_codes, w.w_scales, w.w_zeros, c.w_bits, d_out, c.d_in, s, nt_sub);
  if (c.w_format == EORA_W_SPARSE24_Q4) return launch_repack_sq4(dst, w.w_codes, w.w_scales, w.w_zeros, w.w_meta, d_out, c.d_in, s, nt_sub);
  return launch_repack_sp24(dst, w.w_codes, w.w_zeros, d_out, c.d_in, s, nt_sub);
}

// A view of `m` that starts at row tile t0 (see launch_repack_*).
WMat tile_view(const WMat& m, int t0) {
  WMat v = m;
  v.q = m.q + (int64_t)t0 * m.blob;
  return v;
}

// A view of `m` that starts at pair p0 of the reduction axis and is n_pairs long.
WMat pair_view(const WMat& m, int p0, int n_pairs) {
  WMat v = m;
  v.q = m.q + (int64_t)p0 * m.nt * m.blob;
  v.np = n_pairs; v.kc = 2 * n_pairs; v.k_red = 128 * n_pairs;
  return v;
}

// One backbone with n adapters (decode only): cfg is the layer's, wts[j] carries adapter j (the backbone
// pointers are taken from wts[0]).
int create_multi_impl(const eora_linear_config* cfg, const eora_linear_weights* wts, int n, void* stream, eora_linear_t* out);

// One layer (n == 1) or n layers that share X, stacked along the output axis (fused).
int create_impl(const eora_linear_config* cfgs, const eora_linear_weights* wts, int n, void* stream, eora_linear_t* out) {
  if (out) *out = nullptr;
  if (!cfgs || !wts || !out) return EORA_ERR_NULL_ARG;
  if (n < 1 || n > 4) return EORA_ERR_BAD_SHAPE;
  eora_linear_config c = cfgs[0];
  int d_out_total = 0;
  for (int i = 0; i < n; ++i) {
    int st = check_config(cfgs[i]);
    if (st != EORA_OK) return st;
    st = check_weights(cfgs[i], wts[i]);
    if (st != EORA_OK) return st;
    const eora_linear_config& ci = cfgs[i];
    if (ci.d_in != c.d_in || ci.rank != c.rank || ci.w_format != c.w_format || ci.w_bits != c.w_bits || ci.w_group != c.w_group ||
        ci.ab_format != c.ab_format || ci.ab_group != c.ab_group || ci.x_dtype != c.x_dtype || ci.y_dtype != c.y_dtype ||
        ci.max_m != c.max_m || ci.kernel_policy != c.kernel_policy)
      return EORA_ERR_BAD_SHAPE;
    d_out_total += ci.d_out;
  }
  const bool fused = n > 1;
  if (fused && c.kernel_policy == EORA_POLICY_GENERIC) return EORA_ERR_UNSUPPORTED;
  c.d_out = d_out_total;

  eora_linear* obj = new (std::nothrow) eora_linear();
  if (!obj) return EORA_ERR_CUDA;
  Handle* h = &obj->h;
  *h = Handle();
  h->cfg = c;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  auto fail = [&](int code) {
    if (h->prefill_state) prefill_free(h);
    if (h->tc_state) decode_tc_free(h);
    if (h->stage_mem) cudaFree(h->stage_mem);
    if (h->weight_mem) cudaFree(h->weight_mem);
    if (h->scratch_mem) cudaFree(h->scratch_mem);
    delete obj;
    return code;
  };
  if (cudaGetDevice(&h->device) != cudaSuccess) return fail(EORA_ERR_CUDA);
  if (cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device) != cudaSuccess) return fail(EORA_ERR_CUDA);

  h->wait_limit_ns = 1000000000ull;
  h->r_pad = (int)align_up(c.rank, 128);
  h->n_sub = n;
  h->n_adapters = 1;
  h->t_cols = n * (h->r_pad > 0 ? h->r_pad : 128);
  h->sub_tile0[0] = 0;
  for (int i = 0; i < n; ++i) {
    h->sub_dout[i] = cfgs[i].d_out;
    h->sub_tile0[i + 1] = h->sub_tile0[i] + cfgs[i].d_out / 16;
  }
  for (int i = n + 1; i < 5; ++i) h->sub_tile0[i] = h->sub_tile0[n];
  const bool ab_grouped = c.ab_format == EORA_AB_Q4 || c.ab_format == EORA_AB_Q3;
  int ab_fmt = c.ab_format == EORA_AB_F16 ? FMT_F16 : c.ab_format == EORA_AB_Q4 ? FMT_Q4 : c.ab_format == EORA_AB_Q3 ? FMT_Q3 : FMT_Q8;
  wmat_shape(h->w, backbone_fmt(c), c.d_out, c.d_in, backbone_group(c));
  if (c.rank > 0) {
    int ga = ab_grouped ? c.ab_group : 0;
    int gb = ab_grouped ? (c.ab_group < c.rank ? c.ab_group : c.rank) : 0;
    wmat_shape(h->a, ab_fmt, fused ? n * h->r_pad : c.rank, c.d_in, ga);   // fused: layer i owns rows [i r_pad, (i+1) r_pad)
    wmat_shape(h->b, ab_fmt, c.d_out, h->r_pad, gb);
  } else {
    wmat_shape(h->a, FMT_NONE, 0, 0, 0);
    wmat_shape(h->b, FMT_NONE, 0, 0, 0);
  }

  // ---- weights: one allocation
  Carve sizing{nullptr, 0};
  { WMat tw = h->w, ta = h->a, tb = h->b; wmat_carve(tw, sizing); wmat_carve(ta, sizing); wmat_carve(tb, sizing); }
  h->weight_bytes = sizing.off;
  if (cudaMalloc(&h->weight_mem, (size_t)h->weight_bytes) != cudaSuccess) { h->weight_mem = nullptr; return fail(EORA_ERR_CUDA); }
  Carve wc{reinterpret_cast<char*>(h->weight_mem), 0};
  wmat_carve(h->w, wc); wmat_carve(h->a, wc); wmat_carve(h->b, wc);

  // ---- scratch: one allocation, zero-initialised (the staging buffers of the *_host calls come with the first such call)
  const int64_t rp = h->t_cols;
  bool generic_reachable = c.kernel_policy == EORA_POLICY_GENERIC;
  if (!fused && !generic_reachable) {
    const int probe[8] = {1, 8, 9, 16, 17, 64, 65, c.max_m};
    for (int i = 0; i < 8; ++i)
      if (probe[i] <= c.max_m && !(probe[i] <= 64 && decode_supported(h, probe[i])) && !prefill_supported(h, probe[i])) generic_reachable = true;
  }
  for (int pass = 0; pass < 2; ++pass) {
    Carve sc{reinterpret_cast<char*>(h->scratch_mem), 0};
    // t as fp32 for the simple kernels and as fp16 for the tensor-core family: only where those families can be reached
    h->t_gen = sc.take<float>(generic_reachable ? (int64_t)c.max_m * rp * 4 : 256);
    h->t16 = sc.take<__half>(c.max_m > 8 ? (int64_t)c.max_m * rp * 2 : 256);
    h->d_t = sc.take<float>(8 * rp * 4);
    h->y_ws = sc.take<float>((int64_t)8 * h->w.n_rows * 4);
    h->counters = sc.take<uint32_t>((int64_t)(h->w.nt + 2) * 4);
    h->dev_status = sc.take<int>(256);
    if (pass == 0) {
      h->scratch_bytes = sc.off;
      if (cudaMalloc(&h->scratch_mem, (size_t)h->scratch_bytes) != cudaSuccess) { h->scratch_mem = nullptr; return fail(EORA_ERR_CUDA); }
    }
  }
  if (cudaMemsetAsync(h->scratch_mem, 0, (size_t)h->scratch_bytes, s) != cudaSuccess) return fail(EORA_ERR_CUDA);

  // ---- re-tile, layer by layer into its range of row tiles
  cudaError_t e = cudaSuccess;
  for (int i = 0; i < n && e == cudaSuccess; ++i) {
    const eora_linear_weights& w = wts[i];
    const int d_out_i = cfgs[i].d_out, nt_i = d_out_i / 16;
    const WMat wv = tile_view(h->w, h->sub_tile0[i]);
    e = repack_backbone(wv, c, w, d_out_i, s, fused ? nt_i : -1);
    if (e != cudaSuccess || c.rank == 0) continue;
    const WMat av = tile_view(h->a, fused ? i * h->r_pad / 16 : 0);
    const WMat bv = tile_view(h->b, h->sub_tile0[i]);
    const int a_nt = fused ? h->r_pad / 16 : -1, b_nt = fused ? nt_i : -1;
    if (c.ab_format == EORA_AB_F16) {
      e = launch_repack_f16(av, w.a, c.rank, c.d_in, s, a_nt);
      if (e == cudaSuccess) e = launch_repack_f16(bv, w.b, d_out_i, c.rank, s, b_nt);
    } else if (ab_grouped) {
      const int bits = c.ab_format == EORA_AB_Q4 ? 4 : 3;
      e = launch_repack_quant(av, w.a, w.a_scales, w.a_zeros, bits, c.rank, c.d_in, s, a_nt);
      if (e == cudaSuccess) e = launch_repack_quant(bv, w.b, w.b_scales, w.b_zeros, bits, d_out_i, c.rank, s, b_nt);
    } else {
      e = launch_repack_q8(av, w.a, w.a_scales, w.a_zeros, c.rank, c.d_in, s, a_nt);
      if (e == cudaSuccess) e = launch_repack_q8(bv, w.b, w.b_scales, w.b_zeros, d_out_i, c.rank, s, b_nt);
    }
  }
  if (e != cudaSuccess) return fail(EORA_ERR_CUDA);
  if (prefill_init(h) != cudaSuccess) return fail(EORA_ERR_CUDA);
  if (decode_tc_init(h, s) != cudaSuccess) return fail(EORA_ERR_CUDA);
  if (fused && !decode_supported(h, 1) && !decode_tc_supported(h, 1)) return fail(EORA_ERR_UNSUPPORTED);
  // more than 64 tokens on a fused handle: the tensor-core family only (every layer a whole number of 128-row tiles)
  if (fused && c.max_m > 64 && !prefill_supported(h, c.max_m)) return fail(EORA_ERR_UNSUPPORTED);
  if (cudaStreamSynchronize(s) != cudaSuccess) return fail(EORA_ERR_CUDA);
  *out = obj;
  return EORA_OK;
}

int create_multi_impl(const eora_linear_config* cfg, const eora_linear_weights* wts, int n, void* stream, eora_linear_t* out) {
  if (out) *out = nullptr;
  if (!cfg || !wts || !out) return EORA_ERR_NULL_ARG;
  if (n < 1 || n > 8) return EORA_ERR_BAD_SHAPE;
  const eora_linear_config c = *cfg;
  int st = check_config(c);
  if (st != EORA_OK) return st;
  if (c.rank == 0) return EORA_ERR_BAD_SHAPE;
  if (c.max_m > 64 || c.kernel_policy == EORA_POLICY_GENERIC) return EORA_ERR_UNSUPPORTED;
  for (int j = 0; j < n; ++j) {
    eora_linear_weights w = wts[j];
    w.w_codes = wts[0].w_codes; w.w_scales = wts[0].w_scales; w.w_zeros = wts[0].w_zeros; w.w_meta = wts[0].w_meta;
    st = check_weights(c, w);
    if (st != EORA_OK) return st;
  }

  eora_linear* obj = new (std::nothrow) eora_linear();
  if (!obj) return EORA_ERR_CUDA;
  Handle* h = &obj->h;
  *h = Handle();
  h->cfg = c;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  auto fail = [&](int code) {
    if (h->weight_mem) cudaFree(h->weight_mem);
    if (h->scratch_mem) cudaFree(h->scratch_mem);
    delete obj;
    return code;
  };
  if (cudaGetDevice(&h->device) != cudaSuccess) return fail(EORA_ERR_CUDA);
  if (cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device) != cudaSuccess) return fail(EORA_ERR_CUDA);
  h->wait_limit_ns = 1000000000ull;
  h->r_pad = (int)align_up(c.rank, 128);
  h->n_sub = 1;
  h->n_adapters = n;
  h->multi = 1;
  h->t_cols = n * h->r_pad;
  h->sub_tile0[0] = 0;
  for (int i = 1; i < 5; ++i) h->sub_tile0[i] = c.d_out / 16;
  h->sub_dout[0] = c.d_out;
  const bool ab_grouped = c.ab_format == EORA_AB_Q4 || c.ab_format == EORA_AB_Q3;
  const int ab_fmt = c.ab_format == EORA_AB_F16 ? FMT_F16 : c.ab_format == EORA_AB_Q4 ? FMT_Q4 : c.ab_format == EORA_AB_Q3 ? FMT_Q3 : FMT_Q8;
  wmat_shape(h->w, backbone_fmt(c), c.d_out, c.d_in, backbone_group(c));
  const int ga = ab_grouped ? c.ab_group : 0;
  const int gb = ab_grouped ? (c.ab_group < c.rank ? c.ab_group : c.rank) : 128;   // per-channel: one entry per pair
  wmat_shape(h->a, ab_fmt, n * h->r_pad, c.d_in, ga);
  wmat_shape(h->b, ab_fmt, c.d_out, n * h->r_pad, gb);

  Carve sizing{nullptr, 0};
  { WMat tw = h->w, ta = h->a, tb = h->b; wmat_carve(tw, sizing); wmat_carve(ta, sizing); wmat_carve(tb, sizing); }
  h->weight_bytes = sizing.off;
  if (cudaMalloc(&h->weight_mem, (size_t)h->weight_bytes) != cudaSuccess) { h->weight_mem = nullptr; return fail(EORA_ERR_CUDA); }
  Carve wc{reinterpret_cast<char*>(h->weight_mem), 0};
  wmat_carve(h->w, wc); wmat_carve(h->a, wc); wmat_carve(h->b, wc);

  const int64_t rp = h->t_cols;
  for (int pass = 0; pass < 2; ++pass) {
    Carve sc{reinterpret_cast<char*>(h->scratch_mem), 0};
    h->t_gen = sc.take<float>(256);            // prefill scratch is not used by this kind of handle
    h->t16 = sc.take<__half>(256);
    h->d_t = sc.take<float>(8 * rp * 4);
    h->y_ws = sc.take<float>((int64_t)8 * h->w.n_rows * 4);
    h->counters = sc.take<uint32_t>((int64_t)(h->w.nt + 2) * 4);
    h->dev_status = sc.take<int>(256);
    if (pass == 0) {
      h->scratch_bytes = sc.off;
      if (cudaMalloc(&h->scratch_mem, (size_t)h->scratch_bytes) != cudaSuccess) { h->scratch_mem = nullptr; return fail(EORA_ERR_CUDA); }
    }
  }
  if (cudaMemsetAsync(h->scratch_mem, 0, (size_t)h->scratch_bytes, s) != cudaSuccess) return fail(EORA_ERR_CUDA);

  cudaError_t e = repack_backbone(h->w, c, wts[0], c.d_out, s, -1);
  for (int j = 0; j < n && e == cudaSuccess; ++j) {
    const eora_linear_weights& w = wts[j];
    const WMat av = tile_view(h->a, j * h->r_pad / 16);
    const WMat bv = pair_view(h->b, j * h->r_pad / 128, h->r_pad / 128);
    const int a_nt = h->r_pad / 16;
    if (c.ab_format == EORA_AB_F16) {
      e = launch_repack_f16(av, w.a, c.rank, c.d_in, s, a_nt);
      if (e == cudaSuccess) e = launch_repack_f16(bv, w.b, c.d_out, c.rank, s);
    } else if (ab_grouped) {
      const int bits = c.ab_format == EORA_AB_Q4 ? 4 : 3;
      e = launch_repack_quant(av, w.a, w.a_scales, w.a_zeros, bits, c.rank, c.d_in, s, a_nt);
      if (e == cudaSuccess) e = launch_repack_quant(bv, w.b, w.b_scales, w.b_zeros, bits, c.d_out, c.rank, s);
    } else {
      e = launch_repack_q8(av, w.a, w.a_scales, w.a_zeros, c.rank, c.d_in, s, a_nt);
      if (e == cudaSuccess) e = launch_repack_q8(bv, w.b, w.b_scales, w.b_zeros, c.d_out, c.rank, s);
    }
  }
  if (e != cudaSuccess) return fail(EORA_ERR_CUDA);
  if (!decode_supported(h, 1)) return fail(EORA_ERR_UNSUPPORTED);
  if (cudaStreamSynchronize(s) != cudaSuccess) return fail(EORA_ERR_CUDA);
  *out = obj;
  return EORA_OK;
}

}  // namespace

// Staging buffers of the *_host entry points ([max_m][d_in] activations, [max_m][d_out] results): allocated by the first
// such call on the handle (these calls synchronise anyway), so that handles whose activations live on the device (the
// usual case) do not pay for them.
static int ensure_staging(Handle* h) {
  if (h->stage_mem) return EORA_OK;
  const int64_t xb = align_up((int64_t)h->cfg.max_m * h->cfg.d_in * 2, 256);
  const int64_t yb = align_up((int64_t)h->cfg.max_m * h->cfg.d_out * y_elem_bytes(h->cfg.y_dtype), 256);
  if (cudaMalloc(&h->stage_mem, (size_t)(xb + yb)) != cudaSuccess) { h->stage_mem = nullptr; return EORA_ERR_CUDA; }
  h->stage_bytes = xb + yb;
  h->x_stage = h->stage_mem;
  h->y_stage = reinterpret_cast<char*>(h->stage_mem) + xb;
  return EORA_OK;
}

// The handle's kernels, scratch and shared-memory attributes belong to the device it was created on.
static bool on_handle_device(const Handle* h) {
  int dev = -1;
  return cudaGetDevice(&dev) == cudaSuccess && dev == h->device;
}

extern "C" {

int eora_linear_create(const eora_linear_config* cfg, const eora_linear_weights* wts, void* stream, eora_linear_t* out) {
  return create_impl(cfg, wts, 1, stream, out);
}

int eora_linear_create_fused(const eora_linear_config* cfgs, const eora_linear_weights* wts, int32_t n_layers, void* stream,
                             eora_linear_t* out) {
  return create_impl(cfgs, wts, n_layers, stream, out);
}

int eora_linear_create_multi(const eora_linear_config* cfg, const eora_linear_weights* wts, int32_t n_adapters, void* stream,
                             eora_linear_t* out) {
  return create_multi_impl(cfg, wts, n_adapters, stream, out);
}

int eora_linear_forward_multi(eora_linear_t obj, const void* x, int32_t m, const int32_t* adapter_ids, void* y, void* stream) {
  if (!obj) return EORA_ERR_NULL_ARG;
  if (m == 0) return EORA_OK;
  if (m < 0) return EORA_ERR_BAD_SHAPE;
  if (!x || !y || !adapter_ids) return EORA_ERR_NULL_ARG;
  if (!aligned16(x) || !aligned16(y)) return EORA_ERR_MISALIGNED;
  Handle* h = &obj->h;
  if (!h->multi) return EORA_ERR_UNSUPPORTED;
  if (m > h->cfg.max_m) return EORA_ERR_M_TOO_LARGE;
  if (!on_handle_device(h)) return EORA_ERR_UNSUPPORTED;
  if (!decode_supported(h, m)) return EORA_ERR_UNSUPPORTED;
  void* ys[1] = {y};
  return launch_decode_forward(h, x, m, ys, reinterpret_cast<cudaStream_t>(stream), adapter_ids) == cudaSuccess ? EORA_OK : EORA_ERR_CUDA;
}

int eora_linear_forward_fused(eora_linear_t obj, const void* x, int32_t m, void* const* ys, void* stream) {
  if (!obj) return EORA_ERR_NULL_ARG;
  if (m == 0) return EORA_OK;
  if (m < 0) return EORA_ERR_BAD_SHAPE;
  if (!x || !ys) return EORA_ERR_NULL_ARG;
  Handle* h = &obj->h;
  if (!aligned16(x)) return EORA_ERR_MISALIGNED;
  for (int i = 0; i < h->n_sub; ++i) {
    if (!ys[i]) return EORA_ERR_NULL_ARG;
    if (!aligned16(ys[i])) return EORA_ERR_MISALIGNED;
  }
  if (h->multi) return EORA_ERR_UNSUPPORTED;                  // several adapters: forward_multi says which
  if (m > h->cfg.max_m) return EORA_ERR_M_TOO_LARGE;
  if (!on_handle_device(h)) return EORA_ERR_UNSUPPORTED;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (decode_tc_supported(h, m)) return launch_decode_tc_forward(h, x, m, ys, s) == cudaSuccess ? EORA_OK : EORA_ERR_CUDA;
  if (pick_path(h, m) == EORA_PATH_PREFILL) return launch_prefill_forward(h, x, m, ys, s) == cudaSuccess ? EORA_OK : EORA_ERR_CUDA;
  if (!decode_supported(h, m)) return EORA_ERR_UNSUPPORTED;
  return launch_decode_forward(h, x, m, ys, s) == cudaSuccess ? EORA_OK : EORA_ERR_CUDA;
}

// Device-side alias of a host result buffer the GPU can store to directly (page-locked and mapped), else nullptr. Small
// results are then written by the kernel itself, which saves the copy engine's round trip per output.
static void* mapped_alias(void* host, int32_t m) {
  if (m > 64) return nullptr;                    // large results: the copy engine moves them at full link rate
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, host) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}

// Small activations in mapped page-locked host memory are fetched by a kernel instead of the copy engine: a copy node
// between two launches costs the stream several microseconds (the engine's start and completion, and no overlap with
// the launches around it), a programmatic dependent launch that reads 8-28 KB over the link about two.
__global__ void k_stage_in(const uint4* __restrict__ src, uint4* __restrict__ dst, int64_t n16) {
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");          // the staging buffer may still be read by the launch in front
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n16; i += (int64_t)gridDim.x * blockDim.x) dst[i] = src[i];
}
static int stage_in(Handle* h, const void* x_host, size_t bytes, int32_t m, cudaStream_t s) {
  void* alias = (bytes % 16 == 0 && aligned16(x_host)) ? mapped_alias(const_cast<void*>(x_host), m) : nullptr;
  if (!alias) return cudaMemcpyAsync(h->x_stage, x_host, bytes, cudaMemcpyHostToDevice, s) == cudaSuccess ? EORA_OK : EORA_ERR_CUDA;
  const int64_t n16 = (int64_t)(bytes / 16);
  int grid = (int)((n16 + 1023) / 1024);
  if (grid > 64) grid = 64;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid < 1 ? 1 : grid);
  cfg.blockDim = dim3(256);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_stage_in, reinterpret_cast<const uint4*>(alias), reinterpret_cast<uint4*>(h->x_stage), n16) == cudaSuccess
             ? EORA_OK : EORA_ERR_CUDA;
}

int eora_linear_forward_fused_host_async(eora_linear_t obj, const void* x_host, int32_t m, void* const* ys_host, void* stream) {
  if (!obj) return EORA_ERR_NULL_ARG;
  if (m == 0) return EORA_OK;
  if (m < 0) return EORA_ERR_BAD_SHAPE;
  if (!x_host || !ys_host) return EORA_ERR_NULL_ARG;
  Handle* h = &obj->h;
  for (int i = 0; i < h->n_sub; ++i)
    if (!ys_host[i]) return EORA_ERR_NULL_ARG;
  if (m > h->cfg.max_m) return EORA_ERR_M_TOO_LARGE;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const size_t eb = y_elem_bytes(h->cfg.y_dtype);
  if (h->multi) return EORA_ERR_UNSUPPORTED;
  if (!on_handle_device(h)) return EORA_ERR_UNSUPPORTED;
  if (int rc0 = ensure_staging(h)) return rc0;
  if (int rcs = stage_in(h, x_host, (size_t)m * h->cfg.d_in * 2, m, s)) return rcs;
  void* ys[4] = {nullptr, nullptr, nullptr, nullptr};
  size_t off = 0;
  bool staged[4] = {false, false, false, false};
  for (int i = 0; i < h->n_sub; ++i) {          // staged outputs side by side in the staging buffer ([m][d_out_i] each)
    ys[i] = mapped_alias(ys_host[i], m);
    if (ys[i]) continue;
    staged[i] = true;
    ys[i] = reinterpret_cast<char*>(h->y_stage) + off;
    off += (size_t)m * h->sub_dout[i] * eb;
  }
  int rc = eora_linear_forward_fused(obj, h->x_stage, m, ys, stream);
  if (rc != EORA_OK) return rc;
  for (int i = 0; i < h->n_sub; ++i)
    if (staged[i] && cudaMemcpyAsync(ys_host[i], ys[i], (size_t)m * h->sub_dout[i] * eb, cudaMemcpyDeviceToHost, s) != cudaSuccess) return EORA_ERR_CUDA;
  return EORA_OK;
}

int eora_linear_forward_fused_host(eora_linear_t obj, const void* x_host, int32_t m, void* const* ys_host, void* stream) {
  int rc = eora_linear_forward_fused_host_async(obj, x_host, m, ys_host, stream);
  if (rc != EORA_OK || m == 0) return rc;
  return cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? EORA_OK : EORA_ERR_CUDA;
}

int eora_linear_destroy(eora_linear_t obj) {
  if (!obj) return EORA_OK;
  Handle* h = &obj->h;
  int rc = EORA_OK;
  if (h->prefill_state) prefill_free(h);
  if (h->tc_state) decode_tc_free(h);
  if (h->stage_mem && cudaFree(h->stage_mem) != cudaSuccess) rc = EORA_ERR_CUDA;
  if (h->weight_mem && cudaFree(h->weight_mem) != cudaSuccess) rc = EORA_ERR_CUDA;
  if (h->scratch_mem && cudaFree(h->scratch_mem) != cudaSuccess) rc = EORA_ERR_CUDA;
  delete obj;
  return rc;
}

int eora_linear_path(eora_linear_t obj, int32_t m) {
  if (!obj) return EORA_ERR_NULL_ARG;
  if (m < 1) return EORA_ERR_BAD_SHAPE;
  if (m > obj->h.cfg.max_m) return EORA_ERR_M_TOO_LARGE;
  return pick_path(&obj->h, m);
}

int eora_linear_launches(eora_linear_t obj, int32_t m) {
  int p = eora_linear_path(obj, m);
  if (p < 0) return p;
  if (p == EORA_PATH_DECODE) return decode_tc_supported(&obj->h, m) ? decode_tc_launch_count(&obj->h, m) : decode_launch_count(&obj->h, m);
  if (p == EORA_PATH_PREFILL) return prefill_launch_count(&obj->h, m);
  return generic_launch_count(&obj->h);
}

int eora_linear_forward(eora_linear_t obj, const void* x, int32_t m, void* y, void* stream) {
  if (!obj) return EORA_ERR_NULL_ARG;
  if (m == 0) return EORA_OK;
  if (m < 0) return EORA_ERR_BAD_SHAPE;
  if (!x || !y) return EORA_ERR_NULL_ARG;
  if (!aligned16(x) || !aligned16(y)) return EORA_ERR_MISALIGNED;
  Handle* h = &obj->h;
  if (h->n_sub != 1) return EORA_ERR_UNSUPPORTED;             // fused layers have several outputs: forward_fused
  if (h->multi) return EORA_ERR_UNSUPPORTED;                  // several adapters: forward_multi says which
  if (m > h->cfg.max_m) return EORA_ERR_M_TOO_LARGE;
  if (!on_handle_device(h)) return EORA_ERR_UNSUPPORTED;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  int p = pick_path(h, m);
  cudaError_t e;
  void* ys[1] = {y};
  if (p == EORA_PATH_DECODE) e = decode_tc_supported(h, m) ? launch_decode_tc_forward(h, x, m, ys, s) : launch_decode_forward(h, x, m, ys, s);
  else if (p == EORA_PATH_PREFILL) e = launch_prefill_forward(h, x, m, ys, s);
  else e = launch_generic_forward(h, x, m, y, s);
  return e == cudaSuccess ? EORA_OK : EORA_ERR_CUDA;
}

int eora_linear_forward_host_async(eora_linear_t obj, const void* x_host, int32_t m, void* y_host, void* stream) {
  if (!obj) return EORA_ERR_NULL_ARG;
  if (m == 0) return EORA_OK;
  if (m < 0) return EORA_ERR_BAD_SHAPE;
  if (!x_host || !y_host) return EORA_ERR_NULL_ARG;
  Handle* h = &obj->h;
  if (m > h->cfg.max_m) return EORA_ERR_M_TOO_LARGE;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  size_t xb = (size_t)m * h->cfg.d_in * 2, yb = (size_t)m * h->cfg.d_out * y_elem_bytes(h->cfg.y_dtype);
  if (h->n_sub != 1 || h->multi) return EORA_ERR_UNSUPPORTED;
  if (!on_handle_device(h)) return EORA_ERR_UNSUPPORTED;
  if (int rc0 = ensure_staging(h)) return rc0;
  if (int rcs = stage_in(h, x_host, xb, m, s)) return rcs;
  void* y_dev = mapped_alias(y_host, m);
  int rc = eora_linear_forward(obj, h->x_stage, m, y_dev ? y_dev : h->y_stage, stream);
  if (rc != EORA_OK) return rc;
  if (!y_dev && cudaMemcpyAsync(y_host, h->y_stage, yb, cudaMemcpyDeviceToHost, s) != cudaSuccess) return EORA_ERR_CUDA;
  return EORA_OK;
}

int eora_linear_forward_host(eora_linear_t obj, const void* x_host, int32_t m, void* y_host, void* stream) {
  int rc = eora_linear_forward_host_async(obj, x_host, m, y_host, stream);
  if (rc != EORA_OK || m == 0) return rc;
  return cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? EORA_OK : EORA_ERR_CUDA;
}

int eora_linear_dump(eora_linear_t obj, int32_t what, void* outp, void* stream) {
  if (!obj || !outp) return EORA_ERR_NULL_ARG;
  Handle* h = &obj->h;
  if (what < 0 || what > 3) return EORA_ERR_UNSUPPORTED;
  if (what == 0 && h->cfg.w_format != EORA_W_QUANT) return EORA_ERR_UNSUPPORTED;
  if (what >= 2 && h->cfg.rank == 0) return EORA_ERR_BAD_SHAPE;
  return launch_dump(h, what, outp, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? EORA_OK : EORA_ERR_CUDA;
}

int eora_linear_last_device_status(eora_linear_t obj) {
  if (!obj) return EORA_ERR_NULL_ARG;
  Handle* h = &obj->h;
  int v = 0;
  if (cudaMemcpy(&v, h->dev_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return EORA_ERR_CUDA;
  if (v != 0) {
    // A kernel whose wait ran out returned early and left partial sums, tickets and counters behind: put all
    // scratch that must be zero between launches (status word included) back, so that the handle stays usable.
    char* lo = reinterpret_cast<char*>(h->d_t);
    char* hi = reinterpret_cast<char*>(h->dev_status) + 256;
    if (cudaMemset(lo, 0, (size_t)(hi - lo)) != cudaSuccess) return EORA_ERR_CUDA;
    if (decode_tc_reset(h, nullptr) != cudaSuccess || prefill_reset(h, nullptr) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) return EORA_ERR_CUDA;
  }
  return v;
}

int eora_linear_set_wait_limit(eora_linear_t obj, uint64_t ns) {
  if (!obj) return EORA_ERR_NULL_ARG;
  obj->h.wait_limit_ns = ns ? ns : 1000000000ull;
  return EORA_OK;
}

int eora_linear_selftest_wait_timeout(eora_linear_t obj, void* stream) {
  if (!obj) return EORA_ERR_NULL_ARG;
  if (!on_handle_device(&obj->h)) return EORA_ERR_UNSUPPORTED;
  return launch_wait_selftest(&obj->h, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? EORA_OK : EORA_ERR_CUDA;
}

int64_t eora_linear_staging_bytes(eora_linear_t obj) { return obj ? obj->h.stage_bytes : 0; }

int eora_linear_set_trace(eora_linear_t obj, void* buf) {
  if (!obj) return EORA_ERR_NULL_ARG;
  obj->h.trace = buf;
  return EORA_OK;
}

int eora_linear_decode_grid(eora_linear_t obj, int32_t m) {
  if (!obj) return EORA_ERR_NULL_ARG;
  if (m < 1 || m > 64) return EORA_ERR_BAD_SHAPE;
  if (pick_path(&obj->h, m) != EORA_PATH_DECODE) return 0;
  if (decode_tc_supported(&obj->h, m)) return decode_tc_grid(&obj->h);
  return decode_grid(&obj->h, m);
}

int64_t eora_linear_weight_bytes(eora_linear_t obj) { return obj ? obj->h.weight_bytes + decode_tc_weight_bytes(&obj->h) : 0; }
int64_t eora_linear_scratch_bytes(eora_linear_t obj) { return obj ? obj->h.scratch_bytes + decode_tc_scratch_bytes(&obj->h) : 0; }

}  // extern "C"
