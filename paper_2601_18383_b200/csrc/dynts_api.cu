// Host side of the C ABI declared in include/dynts.h: argument checks, the host mirror of the
// per-sequence lengths, storage layout and kernel launches.  Every step of the path runs in the
// kernels of decode_attn.cuh and evict.cuh; nothing here computes on the CPU.
#include "../../include/dynts.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "common.cuh"
#include "decode_attn.cuh"
#include "decode_stream.cuh"
#include "evict.cuh"
#include "predictor.cuh"
#include "prefill_attn.cuh"

namespace {

thread_local char g_err[512] = "";

dynts_status_t fail(dynts_status_t st, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return st;
}

#define CUDA_TRY(expr)                                                                        \
  do {                                                                                        \
    cudaError_t e_ = (expr);                                                                  \
    if (e_ != cudaSuccess) return fail(DYNTS_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e_)); \
  } while (0)

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {
  size_t K, V, pos, score, comp, agg, src, hdr, len, tot, pinned, target, active, ticket, logit, logit_half, part, arrive, pend, total;
};

// The streaming decode kernel covers bf16 and 8-bit slabs with head_dim 128.
bool stream_capable(const dynts_config_t* c) {
  return (c->dtype == DYNTS_BF16 || c->dtype == DYNTS_BF16_KV8) && c->head_dim == 128 && c->batch <= dynts::kStMaxBatch;
}

int elt_bytes_of(int dtype) { return dtype == DYNTS_FP32 ? 4 : 2; }        // q, k, v, out
int kv_elt_bytes_of(int dtype) { return dtype == DYNTS_BF16_KV8 ? 1 : elt_bytes_of(dtype); }  // slab rows

bool config_ok(const dynts_config_t* c, int* cap_out) {
  if (!c) return false;
  if (c->layers < 1 || c->batch < 1 || c->q_heads < 1 || c->kv_heads < 1 || c->head_dim < 8) return false;
  if (c->q_heads % c->kv_heads) return false;
  if (c->q_heads / c->kv_heads > dynts::kMaxGroup) return false;
  if (c->head_dim % 8 || c->head_dim > 256) return false;
  if (c->dtype != DYNTS_BF16 && c->dtype != DYNTS_FP32 && c->dtype != DYNTS_BF16_KV8) return false;
  if (c->dtype == DYNTS_BF16_KV8 && c->head_dim % 16) return false;  // rows move in 16-byte pieces
  if (c->budget < 1 || c->window < 0 || c->window > c->budget || c->evict_interval < 1) return false;
  int maxb = c->budget;
  if (c->seq_budgets)
    for (int b = 0; b < c->batch; ++b) {
      if (c->seq_budgets[b] < 1 || c->window > c->seq_budgets[b]) return false;
      maxb = std::max(maxb, c->seq_budgets[b]);
    }
  int cap = c->capacity > 0 ? c->capacity : maxb + c->evict_interval;
  if (cap < maxb) return false;
  if (cap_out) *cap_out = cap;
  return true;
}

Layout make_layout(const dynts_config_t* c, int cap) {
  Layout L;
  const size_t slabs = (size_t)c->layers * c->batch * c->kv_heads;
  const size_t kv = slabs * cap * c->head_dim * kv_elt_bytes_of(c->dtype);
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  };
  L.K = take(kv);
  L.V = take(kv);
  L.pos = take(slabs * cap * 4);
  L.score = take(slabs * cap * 4);
  L.comp = take(slabs * cap * 4);
  L.agg = take((size_t)c->batch * cap * 4);
  L.src = take(slabs * cap * 4);
  L.hdr = take(slabs * 16);
  L.len = take((size_t)c->batch * 4);
  L.tot = take((size_t)c->batch * 4);
  L.pinned = take((size_t)c->batch * 4);
  L.target = take((size_t)c->batch * 4);
  L.active = take((size_t)c->batch * 4);
  L.ticket = take(256);
  L.logit = L.part = L.arrive = L.pend = off;
  L.logit_half = 0;
  if (stream_capable(c)) {
    // two halves: a step writes one while the recorded score passes of the step before read the other
    L.logit_half = align_up(slabs * (size_t)(c->q_heads / c->kv_heads) * cap * 4, 256);
    L.logit = take(2 * L.logit_half);
    L.part = take((size_t)dynts::kStMaxCtas * 2 * dynts::kStPartStride * 4);
    L.arrive = take(slabs * 4);
    L.pend = take(slabs * (size_t)dynts::kStPendWords * 4);
  }
  L.total = off;
  return L;
}

}  // namespace

struct dynts_cache {
  dynts_config_t cfg;
  int cap = 0;
  int G = 1;
  int elt = 2;               // bytes per element of q, k, v, out
  int kv_elt = 2;            // bytes per element of the slab rows
  float k_scale = 1.f, v_scale = 1.f;  // 8-bit slabs: stored code = e4m3(x / scale)
  bool ready = false;        // storage exists
  bool owns_storage = false;
  char* base = nullptr;
  Layout lay{};
  cudaStream_t stream = nullptr;
  int* err_host = nullptr;   // pinned, mapped
  int* err_dev = nullptr;
  std::vector<int> seq_budget, len_h, tot_h, pinned_h, target_h, active_h;  // host mirrors of the per-sequence state
  int layer_cursor = 0;      // next layer expected by dynts_decode_attn_layer
  int cluster = 0, variant = 0;
  unsigned int wait_limit = dynts::kStSpinLimit;  // polls of a bounded device-side wait
  int drop_item = -1;        // one-shot: the next streaming decode launch omits this tile load of CTA 0 (timeout-path test)
  int evict_split = 0;       // CTAs per slab of the eviction: 0 automatic, 1/2/4/8 forced, -1 the one-CTA kernel with shared-memory keys
  int score_source = 0;      // 0: attention mass accumulates (Eq. 6); 1: the caller supplies scores (Eq. 7)
  int parity = 0;            // half of the logit scratch the next decode step writes
  bool pending = false;      // the last streaming launches recorded score passes that are not applied yet
  long long launches = 0;
  // staging for the host-buffer entry point
  char* stage_dev = nullptr;
  size_t stage_bytes = 0;
  bool attr_generic_f32 = false, attr_generic_bf16 = false, attr_generic_kv8 = false, attr_mma = false, attr_select = false;
  bool attr_stream = false, attr_fused = false, attr_prefill = false;
  bool have_maps = false;    // tensor maps of the K and V slabs for the streaming kernel
  CUtensorMap map_KV;
  int sm_count = 0;

  void* K() const { return base + lay.K; }
  void* V() const { return base + lay.V; }
  int* pos() const { return reinterpret_cast<int*>(base + lay.pos); }
  float* score() const { return reinterpret_cast<float*>(base + lay.score); }
  float* comp() const { return reinterpret_cast<float*>(base + lay.comp); }
  float* agg() const { return reinterpret_cast<float*>(base + lay.agg); }
  int* src() const { return reinterpret_cast<int*>(base + lay.src); }
  int* hdr() const { return reinterpret_cast<int*>(base + lay.hdr); }
  int* len() const { return reinterpret_cast<int*>(base + lay.len); }
  int* tot() const { return reinterpret_cast<int*>(base + lay.tot); }
  int* pinned() const { return reinterpret_cast<int*>(base + lay.pinned); }
  int* target() const { return reinterpret_cast<int*>(base + lay.target); }
  int* active() const { return reinterpret_cast<int*>(base + lay.active); }
  unsigned int* ticket() const { return reinterpret_cast<unsigned int*>(base + lay.ticket); }
  float* logit(int half) const { return reinterpret_cast<float*>(base + lay.logit + (size_t)half * lay.logit_half); }
  int* pend() const { return reinterpret_cast<int*>(base + lay.pend); }
  float* part() const { return reinterpret_cast<float*>(base + lay.part); }
  int* arrive() const { return reinterpret_cast<int*>(base + lay.arrive); }
  size_t slabs() const { return (size_t)cfg.layers * cfg.batch * cfg.kv_heads; }
};

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Tensor map (TMA descriptor) over all K rows and all V rows, read in boxes of 32 rows with the
// 128-byte shared-memory swizzle.
typedef CUresult (*tensor_map_encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                         const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                         CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

dynts_status_t make_slab_maps(dynts_cache* c) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
  if (!fn || qres != cudaDriverEntryPointSuccess) return fail(DYNTS_ERR_CUDA, "the driver has no cuTensorMapEncodeTiled");
  tensor_map_encode_fn encode = reinterpret_cast<tensor_map_encode_fn>(fn);
  const cuuint64_t rows = (cuuint64_t)c->slabs() * c->cap;
  if (rows >= ((cuuint64_t)1 << 31)) return DYNTS_OK;  // row coordinates are 32-bit: keep the cluster kernels
  // One map over both tensors, [2 (K, V)][slabs * cap rows][128 elements], so that one tile load
  // brings the K box and the V box of a chunk.  bf16 rows: 256 bytes read as boxes of 64 elements;
  // 8-bit rows: 128 bytes, one box of 128 codes.
  const bool kv8 = c->cfg.dtype == DYNTS_BF16_KV8;
  const cuuint64_t kv_stride = (cuuint64_t)(static_cast<char*>(c->V()) - static_cast<char*>(c->K()));
  if (kv_stride == 0 || (kv_stride & 15u) != 0 || kv_stride >= ((cuuint64_t)1 << 40)) return DYNTS_OK;  // keep the cluster kernels
  const cuuint64_t dims[3] = {128, rows, 2};
  const cuuint64_t strides[2] = {kv8 ? 128u : 256u, kv_stride};
  const cuuint32_t box[3] = {kv8 ? 128u : 64u, (cuuint32_t)dynts::kStRows, 2};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUtensorMapDataType mtype = kv8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  CUresult r1 = encode(&c->map_KV, mtype, 3, c->K(), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                       CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r1 != CUDA_SUCCESS) return fail(DYNTS_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r1);
  c->have_maps = true;
  return DYNTS_OK;
}

dynts_status_t materialise(dynts_cache* c) {
  if (c->ready) return DYNTS_OK;
  int cap = 0;
  if (!config_ok(&c->cfg, &cap)) return fail(DYNTS_ERR_INVALID_ARG, "invalid cache configuration");
  c->cap = cap;
  c->G = c->cfg.q_heads / c->cfg.kv_heads;
  c->elt = elt_bytes_of(c->cfg.dtype);
  c->kv_elt = kv_elt_bytes_of(c->cfg.dtype);
  c->lay = make_layout(&c->cfg, cap);
  if (c->cfg.storage) {
    if ((reinterpret_cast<uintptr_t>(c->cfg.storage) & 255u) != 0)
      return fail(DYNTS_ERR_INVALID_ARG, "storage must be 256-byte aligned");
    if (c->cfg.storage_bytes < c->lay.total)
      return fail(DYNTS_ERR_OOM, "storage too small: %zu < %zu bytes", c->cfg.storage_bytes, c->lay.total);
    c->base = static_cast<char*>(c->cfg.storage);
    c->owns_storage = false;
  } else {
    void* p = nullptr;
    cudaError_t e = cudaMalloc(&p, c->lay.total);
    if (e != cudaSuccess) return fail(DYNTS_ERR_OOM, "cudaMalloc(%zu): %s", c->lay.total, cudaGetErrorString(e));
    c->base = static_cast<char*>(p);
    c->owns_storage = true;
  }
  if (!c->err_host) {
    cudaError_t e = cudaHostAlloc(reinterpret_cast<void**>(&c->err_host), 64, cudaHostAllocMapped);
    if (e != cudaSuccess) return fail(DYNTS_ERR_OOM, "cudaHostAlloc: %s", cudaGetErrorString(e));
    *c->err_host = 0;
    CUDA_TRY(cudaHostGetDevicePointer(reinterpret_cast<void**>(&c->err_dev), c->err_host, 0));
  }
  CUDA_TRY(cudaMemsetAsync(c->base, 0, c->lay.total, c->stream));
  {
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    CUDA_TRY(cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev));
  }
  c->have_maps = false;
  if (stream_capable(&c->cfg)) {
    dynts_status_t ms = make_slab_maps(c);
    if (ms != DYNTS_OK) return ms;
  }
  const int Nb = c->cfg.batch;
  c->seq_budget.assign(Nb, c->cfg.budget);
  if (c->cfg.seq_budgets)
    for (int b = 0; b < Nb; ++b) c->seq_budget[b] = c->cfg.seq_budgets[b];
  c->cfg.seq_budgets = nullptr;  // the caller's array is not kept
  c->len_h.assign(Nb, 0);
  c->tot_h.assign(Nb, 0);
  c->pinned_h.assign(Nb, 0);
  c->active_h.assign(Nb, 1);
  c->target_h = c->seq_budget;
  CUDA_TRY(cudaMemcpyAsync(c->target(), c->target_h.data(), Nb * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(cudaMemcpyAsync(c->active(), c->active_h.data(), Nb * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(cudaStreamSynchronize(c->stream));  // the host vectors above may be reused right away
  c->ready = true;
  return DYNTS_OK;
}

template <typename Kern>
dynts_status_t ensure_smem_attr(Kern kern, size_t bytes, bool* done, bool nonportable) {
  if (!*done) {
    CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    if (nonportable) CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
    *done = true;
  }
  if (bytes > 200 * 1024) return fail(DYNTS_ERR_INVALID_ARG, "shared-memory need %zu exceeds 200 KiB", bytes);
  return DYNTS_OK;
}

int pick_cluster(const dynts_cache* c, int units, int n_max) {
  if (c->cluster > 0) return c->cluster;
  // Enough CTAs to fill 148 SMs several times over, but at least ~64 rows per CTA.
  int s = 1;
  while (s < 8 && (long long)units * s < 148 * 6 && n_max / (2 * s) >= 64) s *= 2;
  return s;
}

// Applies the score passes that streaming launches left recorded (DecodeParams::defer).  Called
// before anything but the next deferring decode launch reads or writes the scores.
dynts_status_t flush_pending(dynts_cache* c) {
  if (!c->pending) return DYNTS_OK;
  cudaLaunchConfig_t fc;
  memset(&fc, 0, sizeof(fc));
  cudaLaunchAttribute fattr[1];
  fattr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see griddepcontrol.wait in the kernel
  fattr[0].val.programmaticStreamSerializationAllowed = 1;
  fc.attrs = fattr;
  fc.numAttrs = 1;
  fc.stream = c->stream;
  fc.gridDim = dim3((unsigned)c->slabs(), 1, 1);
  fc.blockDim = dim3(128, 1, 1);
  CUDA_TRY(cudaLaunchKernelEx(&fc, dynts::flush_pending_kernel, c->score(), c->comp(), (const float*)c->logit(c->parity ^ 1),
                              c->pend(), c->G, c->cap));
  c->launches += 1;
  c->pending = false;
  return DYNTS_OK;
}

dynts_status_t launch_decode(dynts_cache* c, int layer0, int n_layers, const void* q, const void* k_new,
                             const void* v_new, void* out, float* scores, bool advance) {
  const dynts_config_t& f = c->cfg;
  const int Nb = f.batch;
  int n_max = 0;
  bool any = false;
  for (int b = 0; b < Nb; ++b) {
    if (!c->active_h[b]) continue;
    any = true;
    if (c->len_h[b] + 1 > c->cap)
      return fail(DYNTS_ERR_CAPACITY, "sequence %d is at capacity %d: evict before the next decode step", b, c->cap);
    n_max = std::max(n_max, c->len_h[b] + 1);
  }
  if (!any) return DYNTS_OK;

  const int units = n_layers * Nb * f.kv_heads;
  const int S = pick_cluster(c, units, n_max);
  const int units16 = (n_max + 15) / 16;
  const int tile_tokens = (units16 + S - 1) / S * 16;

  dynts::DecodeParams p;
  p.q = q;
  p.k_new = k_new;
  p.v_new = v_new;
  p.out = out;
  p.delta_out = scores;
  p.K = c->K();
  p.V = c->V();
  p.pos = c->pos();
  p.score = c->score();
  p.comp = c->comp();
  p.len = c->len();
  p.tot = c->tot();
  p.active = c->active();
  p.ticket = c->ticket();
  p.err = c->err_dev;
  p.logit = c->logit(c->parity);
  p.logit_prev = c->logit(c->parity ^ 1);
  p.pend = c->pend();
  p.defer = 0;
  p.part = c->part();
  p.arrive = c->arrive();
  p.dbg = reinterpret_cast<int*>(c->ticket()) + 8;  // spare words of the ticket block
  p.layer0 = layer0;
  p.n_layers = n_layers;
  p.Nb = Nb;
  p.Hkv = f.kv_heads;
  p.G = c->G;
  p.d = f.head_dim;
  p.cap = c->cap;
  p.advance = advance ? 1 : 0;
  p.tile_tokens = tile_tokens;
  p.slabs_per_cta = 0;
  p.accumulate = c->score_source == 0 ? 1 : 0;
  p.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)f.head_dim));
  p.k_scale = c->k_scale;
  p.v_scale = c->v_scale;
  p.out_scale = 1.f;
  const bool kv8 = f.dtype == DYNTS_BF16_KV8;
  if (kv8) {
    p.scale_log2 *= c->k_scale;
    p.out_scale = c->v_scale;
  }

  // Lengths with the launch (streaming kernel): not while the stream is being captured, since a
  // replayed graph would carry the lengths of the capture.
  p.spin_limit = c->wait_limit;
  p.drop_item = -1;
  p.n_host = 0;
  if (Nb <= dynts::kHostLens) {
    cudaStreamCaptureStatus cap_status = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(c->stream, &cap_status) == cudaSuccess && cap_status == cudaStreamCaptureStatusNone) {
      p.n_host = Nb;
      for (int b = 0; b < dynts::kHostLens; ++b) {
        p.len_host[b] = (b < Nb && c->active_h[b]) ? c->len_h[b] : -1;
        p.tot_host[b] = b < Nb ? c->tot_h[b] : 0;
      }
    }
  }
  const bool mma_ok = f.dtype == DYNTS_BF16 && f.head_dim == 128 && c->G <= 8;
  const bool stream_ok = (mma_ok || (kv8 && f.head_dim == 128 && c->G <= 8)) && c->have_maps;
  int variant = c->variant;
  if (variant == 0) variant = stream_ok ? 3 : (mma_ok ? 2 : 1);
  if (variant == 2 && kv8) variant = 1;  // the cluster tensor-core kernel reads bf16 rows only
  if (variant == 2 && !mma_ok) return fail(DYNTS_ERR_INVALID_ARG, "tensor-core variant needs bf16, head_dim 128, G <= 8");
  if (variant == 3 && !stream_ok)
    return fail(DYNTS_ERR_INVALID_ARG, "streaming variant needs bf16 or 8-bit slabs, head_dim 128, G <= 8, batch <= %d",
                dynts::kStMaxBatch);

  if (variant == 3) {
    const size_t smem = dynts::stream_smem_bytes(Nb);
    if (!c->attr_stream) {
      const int smem_max = (int)dynts::stream_smem_bytes(dynts::kStMaxBatch);
      if (kv8) {
        CUDA_TRY(cudaFuncSetAttribute(dynts::decode_attn_stream_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max));
        CUDA_TRY(cudaFuncSetAttribute(dynts::decode_attn_stream_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max));
      } else {
        CUDA_TRY(cudaFuncSetAttribute(dynts::decode_attn_stream_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max));
      }
      c->attr_stream = true;
    }
    int ctas = ((c->cluster == 1 || c->cluster == 2) ? c->cluster : 2) * c->sm_count;
    ctas = std::max(1, std::min(ctas, dynts::kStMaxCtas));
    // Equally long slabs and at least about as many slabs as CTAs: give every CTA whole slabs, so
    // that no slab needs the cross-CTA combine.  Otherwise the chunk list is cut into equal pieces.
    p.slabs_per_cta = 0;
    {
      bool uniform = true;
      int n_active = 0, len0 = -1;
      for (int b = 0; b < Nb; ++b) {
        if (!c->active_h[b]) continue;
        ++n_active;
        if (len0 < 0) len0 = c->len_h[b];
        uniform = uniform && c->len_h[b] == len0;
      }
      const long long slabs = (long long)n_layers * n_active * f.kv_heads;
      const long long per = (slabs + ctas - 1) / ctas;
      const long long used = (slabs + per - 1) / per;
      // (bf16 slabs: the launch is HBM-bound, so 80 % of the CTA slots are enough and the combine is
      // what one saves; 8-bit slabs: a CTA's own pipeline bounds it, so idle slots cost throughput
      // unless the launch is so short -- a slab or two per CTA -- that the combine would cost more)
      const bool mostly = used * 5 >= (long long)ctas * 4, nearly_all = used * 20 >= (long long)ctas * 19;
      if (uniform && (kv8 ? (nearly_all || (mostly && per <= 2)) : mostly)) {
        p.slabs_per_cta = (int)per;
        ctas = (int)used;
      } else if (!kv8 && c->cluster == 0 && slabs <= c->sm_count) {
        // Fewer slabs than SMs (one layer of a small batch): every slab is shared by several CTAs
        // however the list is cut.  One CTA per SM then halves the partial results per slab, and
        // the CTAs of the next launch in the stream find room to become resident and run their
        // set-up during this launch's tail.  (64 slabs of 3080 rows: 31.0 us per launch against
        // 34.3 us with two CTAs per SM, the best of 64..296 CTAs; 116 against 133 us at 16500
        // rows; from 192 slabs on two per SM are faster again.)
        ctas = std::min(ctas, c->sm_count);
      }
    }
    // The score pass of every CTA's last slab moves into the next launch when the pieces are whole
    // slabs, the lengths travel with the launch (so the piece shape is certain), the scores
    // accumulate and nobody asked for this step's mass.
    // (Only launches that cover all layers: the records of a step then sit in one half of the scratch.)
    const bool defer = n_layers == f.layers && p.slabs_per_cta > 0 && p.n_host > 0 && p.accumulate && scores == nullptr;
    if (!defer) {
      dynts_status_t fs = flush_pending(c);
      if (fs != DYNTS_OK) return fs;
    }
    p.defer = defer ? 1 : 0;
    p.drop_item = c->drop_item;
    c->drop_item = -1;
    auto* stream_kernel = !kv8 ? dynts::decode_attn_stream_kernel<false, true>
                               : (defer ? dynts::decode_attn_stream_kernel<true, true> : dynts::decode_attn_stream_kernel<true, false>);
    cudaLaunchConfig_t sc;
    memset(&sc, 0, sizeof(sc));
    cudaLaunchAttribute sattr[1];
    sattr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see griddepcontrol.wait in the kernel
    sattr[0].val.programmaticStreamSerializationAllowed = 1;
    sc.attrs = sattr;
    sc.numAttrs = 1;
    sc.stream = c->stream;
    sc.gridDim = dim3((unsigned)ctas, 1, 1);
    sc.blockDim = dim3(dynts::kStThreads, 1, 1);
    sc.dynamicSmemBytes = smem;
    cudaError_t e = cudaLaunchKernelEx(&sc, stream_kernel, p, c->map_KV);
    if (e != cudaSuccess) return fail(DYNTS_ERR_CUDA, "decode launch (streaming, %d CTAs): %s", ctas, cudaGetErrorString(e));
    c->launches += 1;
    if (defer) c->pending = true;
    if (advance) {
      if (defer) c->parity ^= 1;  // the next step must not overwrite the logits of the recorded passes
      for (int b = 0; b < Nb; ++b)
        if (c->active_h[b]) {
          c->len_h[b] += 1;
          c->tot_h[b] += 1;
        }
    }
    return DYNTS_OK;
  }
  {
    dynts_status_t fs = flush_pending(c);  // the cluster kernels update the scores themselves
    if (fs != DYNTS_OK) return fs;
  }

  cudaLaunchConfig_t lc;
  memset(&lc, 0, sizeof(lc));
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = S;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  lc.attrs = attr;
  lc.numAttrs = 1;
  lc.stream = c->stream;
  lc.gridDim = dim3((unsigned)(units * S), 1, 1);

  cudaError_t e;
  if (variant == 2) {
    const size_t smem = dynts::mma_smem_bytes(c->G, tile_tokens);
    dynts_status_t st = ensure_smem_attr(dynts::decode_attn_mma_kernel, smem, &c->attr_mma, true);
    if (st != DYNTS_OK) return st;
    lc.blockDim = dim3(dynts::kMmaThreads, 1, 1);
    lc.dynamicSmemBytes = smem;
    e = cudaLaunchKernelEx(&lc, dynts::decode_attn_mma_kernel, p);
  } else if (kv8) {
    const size_t smem = dynts::generic_smem_bytes(c->G, f.head_dim, tile_tokens);
    dynts_status_t st =
        ensure_smem_attr(dynts::decode_attn_generic_kernel<__nv_bfloat16, true>, smem, &c->attr_generic_kv8, true);
    if (st != DYNTS_OK) return st;
    lc.blockDim = dim3(dynts::kGenericThreads, 1, 1);
    lc.dynamicSmemBytes = smem;
    e = cudaLaunchKernelEx(&lc, dynts::decode_attn_generic_kernel<__nv_bfloat16, true>, p);
  } else if (f.dtype == DYNTS_FP32) {
    const size_t smem = dynts::generic_smem_bytes(c->G, f.head_dim, tile_tokens);
    dynts_status_t st = ensure_smem_attr(dynts::decode_attn_generic_kernel<float>, smem, &c->attr_generic_f32, true);
    if (st != DYNTS_OK) return st;
    lc.blockDim = dim3(dynts::kGenericThreads, 1, 1);
    lc.dynamicSmemBytes = smem;
    e = cudaLaunchKernelEx(&lc, dynts::decode_attn_generic_kernel<float>, p);
  } else {
    const size_t smem = dynts::generic_smem_bytes(c->G, f.head_dim, tile_tokens);
    dynts_status_t st =
        ensure_smem_attr(dynts::decode_attn_generic_kernel<__nv_bfloat16>, smem, &c->attr_generic_bf16, true);
    if (st != DYNTS_OK) return st;
    lc.blockDim = dim3(dynts::kGenericThreads, 1, 1);
    lc.dynamicSmemBytes = smem;
    e = cudaLaunchKernelEx(&lc, dynts::decode_attn_generic_kernel<__nv_bfloat16>, p);
  }
  if (e != cudaSuccess) return fail(DYNTS_ERR_CUDA, "decode launch (cluster %d): %s", S, cudaGetErrorString(e));
  c->launches += 1;
  if (advance)
    for (int b = 0; b < Nb; ++b)
      if (c->active_h[b]) {
          c->len_h[b] += 1;
          c->tot_h[b] += 1;
        }
  return DYNTS_OK;
}

dynts_status_t check_decode_args(const dynts_cache* c, const void* q, const void* k_new, const void* v_new,
                                 const void* out) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (!q || !k_new || !v_new || !out) return fail(DYNTS_ERR_INVALID_ARG, "NULL tensor pointer");
  if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out))
    return fail(DYNTS_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned");
  return DYNTS_OK;
}

// layer < 0: all layers (k, v hold L layers); else that one layer (k, v hold one), the lengths being
// published with the last layer.
dynts_status_t do_prefill(dynts_cache* c, int seq, const void* k, const void* v, int T, int n_pinned, int layer = -1) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  dynts_status_t st = materialise(c);
  if (st != DYNTS_OK) return st;
  if (!k || !v || !aligned16(k) || !aligned16(v))
    return fail(DYNTS_ERR_INVALID_ARG, "prefill tensors must be non-NULL and 16-byte aligned");
  if (T < 0 || T > c->cap) return fail(DYNTS_ERR_CAPACITY, "prefill of %d rows exceeds capacity %d", T, c->cap);
  if (n_pinned < 0 || n_pinned > T) return fail(DYNTS_ERR_INVALID_ARG, "n_pinned %d outside [0, %d]", n_pinned, T);
  if (seq >= c->cfg.batch) return fail(DYNTS_ERR_INVALID_ARG, "sequence %d out of range", seq);
  if (c->layer_cursor != 0) return fail(DYNTS_ERR_STATE, "prefill in the middle of a layer-by-layer step");
  {
    dynts_status_t fs_ = flush_pending(c);
    if (fs_ != DYNTS_OK) return fs_;
  }
  dynts::PrefillParams p;
  p.k = k;
  p.v = v;
  p.K = c->K();
  p.V = c->V();
  p.pos = c->pos();
  p.score = c->score();
  p.comp = c->comp();
  p.len = c->len();
  p.tot = c->tot();
  p.pinned = c->pinned();
  p.active = c->active();
  p.L = c->cfg.layers;
  p.Nb = c->cfg.batch;
  p.Hkv = c->cfg.kv_heads;
  p.d = c->cfg.head_dim;
  p.cap = c->cap;
  p.elt_bytes = c->kv_elt;
  p.kv8 = c->cfg.dtype == DYNTS_BF16_KV8 ? 1 : 0;
  p.k_scale = c->k_scale;
  p.v_scale = c->v_scale;
  p.T = T;
  p.n_pinned = n_pinned;
  p.seq = seq;
  const int n_layers = layer < 0 ? c->cfg.layers : 1;
  const bool publish = layer < 0 || layer == c->cfg.layers - 1;
  p.layer0 = layer < 0 ? 0 : layer;
  p.set_len = publish ? 1 : 0;
  const unsigned ny = (unsigned)((size_t)n_layers * (seq < 0 ? c->cfg.batch : 1) * c->cfg.kv_heads);
  const size_t pieces = (size_t)T * c->cfg.head_dim * c->elt / 16;  // 16-byte pieces of the source
  const unsigned nx = (unsigned)std::max<size_t>(1, std::min<size_t>(64, (pieces + 255) / 256));
  dynts::prefill_kernel<<<dim3(nx, ny, 1), 256, 0, c->stream>>>(p);
  CUDA_TRY(cudaGetLastError());
  c->launches += 1;
  for (int b = 0; b < c->cfg.batch && publish; ++b) {
    if (seq >= 0 && b != seq) continue;
    c->len_h[b] = T;
    c->tot_h[b] = T;
    c->pinned_h[b] = n_pinned;
    c->active_h[b] = 1;
  }
  return DYNTS_OK;
}

dynts_status_t do_evict(dynts_cache* c, const int* targets /* host [Nb], validated */, bool global = false) {
  // Recorded score passes: the fused kernel applies them slab by slab before it reads the scores;
  // the other paths (aggregated keys, very long slabs) need them applied beforehand.
  const bool fused_path = c->cap <= (global ? 10000 : 12800);  // (the shared keys take a fifth array of the CTA's shared memory)
  if (global || !fused_path) {
    dynts_status_t fs_ = flush_pending(c);
    if (fs_ != DYNTS_OK) return fs_;
  }
  const int Nb = c->cfg.batch;
  bool any = false;
  for (int b = 0; b < Nb; ++b) {
    if (!c->active_h[b] || c->len_h[b] <= targets[b]) continue;
    if (c->pinned_h[b] + c->cfg.window > targets[b])
      return fail(DYNTS_ERR_BUDGET, "sequence %d: question window %d + local window %d exceed target %d", b,
                  c->pinned_h[b], c->cfg.window, targets[b]);
    any = true;
  }
  if (!any) return DYNTS_OK;
  bool same = true;
  for (int b = 0; b < Nb; ++b) same = same && c->target_h[b] == targets[b];
  if (!same) {
    c->target_h.assign(targets, targets + Nb);
    // pageable source: the runtime stages it before returning, so target_h may change afterwards
    CUDA_TRY(cudaMemcpyAsync(c->target(), c->target_h.data(), Nb * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  }
  dynts::EvictParams p;
  p.K = c->K();
  p.V = c->V();
  p.pos = c->pos();
  p.score = c->score();
  p.comp = c->comp();
  p.key = nullptr;
  p.src = c->src();
  p.hdr = c->hdr();
  p.len = c->len();
  p.pinned = c->pinned();
  p.target = c->target();
  p.err = c->err_dev;
  p.L = c->cfg.layers;
  p.Nb = Nb;
  p.Hkv = c->cfg.kv_heads;
  p.d = c->cfg.head_dim;
  p.cap = c->cap;
  p.window = c->cfg.window;
  p.elt_bytes = c->kv_elt;
  if (global) {
    // one score per token: sum the slab scores of each sequence, every slab then ranks by the sum
    dynts::aggregate_scores_kernel<<<dim3((unsigned)((c->cap + 255) / 256), (unsigned)Nb, 1), 256, 0, c->stream>>>(
        c->score(), c->agg(), c->len(), c->active(), c->cfg.layers, Nb, c->cfg.kv_heads, c->cap);
    CUDA_TRY(cudaGetLastError());
    c->launches += 1;
    p.key = c->agg();
  }
  if (fused_path) {
    // one launch: selection and compaction of a slab by the same CTA, or by a cluster of CTAs that
    // share the slab's columns
    if (c->pending) {
      p.pend = c->pend();
      p.logit_prev = c->logit(c->parity ^ 1);
      p.G = c->G;
      c->pending = false;
    }
    cudaLaunchConfig_t fc;
    memset(&fc, 0, sizeof(fc));
    cudaLaunchAttribute fattr[2];
    fattr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see griddepcontrol.wait in the kernel
    fattr[0].val.programmaticStreamSerializationAllowed = 1;
    fc.attrs = fattr;
    fc.numAttrs = 1;
    fc.stream = c->stream;
    const int pieces2 = 2 * c->cfg.head_dim * c->kv_elt / 16;  // 16-byte pieces of a K row followed by a V row
    // Slabs of up to 2304 rows: the kernel that keeps a thread's rows in registers (its short
    // selection phase matters there); longer slabs, whose events are dominated by the rows that
    // move, measured faster on the one-CTA kernel with shared-memory keys.
    if (c->cap <= 17 * dynts::kSplitThreads && (c->evict_split > 0 || (c->evict_split == 0 && c->cap <= 9 * dynts::kSplitThreads))) {
      // CTAs per slab: as many as still leave every CTA of the grid resident at once (a second round
      // of CTAs would start only when the first ends), in shares of at least 64 contiguous bytes
      const int tier = c->cap <= 5 * dynts::kSplitThreads ? 5 : c->cap <= 9 * dynts::kSplitThreads ? 9 : c->cap <= 13 * dynts::kSplitThreads ? 13 : 17;
      const long long resident = (long long)(c->sm_count > 0 ? c->sm_count : 148) * dynts::split_ctas_per_sm(tier);
      int S = 1;
      if (c->evict_split > 0) {
        S = c->evict_split;
      } else {
        while (S < 8 && (long long)c->slabs() * (2 * S) <= resident) S *= 2;
      }
      while (S > 1 && (pieces2 % S != 0 || pieces2 / S < 4)) S /= 2;
      fattr[1].id = cudaLaunchAttributeClusterDimension;
      fattr[1].val.clusterDim.x = (unsigned)S;
      fattr[1].val.clusterDim.y = 1;
      fattr[1].val.clusterDim.z = 1;
      fc.numAttrs = 2;
      fc.gridDim = dim3((unsigned)(c->slabs() * S), 1, 1);
      fc.blockDim = dim3(dynts::kSplitThreads, 1, 1);
      fc.dynamicSmemBytes = (size_t)c->cap * 4;
      cudaError_t e;
#define DYNTS_SPLIT_LAUNCH(RPT)                                                                                   \
  (global ? cudaLaunchKernelEx(&fc, dynts::evict_split_kernel<RPT, true>, p, c->ticket() + 1)                     \
          : cudaLaunchKernelEx(&fc, dynts::evict_split_kernel<RPT, false>, p, c->ticket() + 1))
      if (tier == 5) e = DYNTS_SPLIT_LAUNCH(5);
      else if (tier == 9) e = DYNTS_SPLIT_LAUNCH(9);
      else if (tier == 13) e = DYNTS_SPLIT_LAUNCH(13);
      else e = DYNTS_SPLIT_LAUNCH(17);
#undef DYNTS_SPLIT_LAUNCH
      if (e != cudaSuccess) return fail(DYNTS_ERR_CUDA, "eviction launch (%d CTAs per slab): %s", S, cudaGetErrorString(e));
    } else {
      const size_t smem = (size_t)c->cap * (global ? 20 : 16);
      dynts_status_t st = ensure_smem_attr(dynts::evict_fused_kernel, smem, &c->attr_fused, false);
      if (st != DYNTS_OK) return st;
      fc.gridDim = dim3((unsigned)c->slabs(), 1, 1);
      fc.blockDim = dim3(dynts::kFusedThreads, 1, 1);
      fc.dynamicSmemBytes = smem;
      CUDA_TRY(cudaLaunchKernelEx(&fc, dynts::evict_fused_kernel, p, c->ticket() + 1));
    }
    c->launches += 1;
  } else {
    const size_t smem = (size_t)c->cap * 12;
    dynts_status_t st = ensure_smem_attr(dynts::evict_select_kernel, smem, &c->attr_select, false);
    if (st != DYNTS_OK) return st;
    dynts::evict_select_kernel<<<(unsigned)c->slabs(), dynts::kSelectThreads, smem, c->stream>>>(p);
    CUDA_TRY(cudaGetLastError());
    const int pieces = c->cfg.head_dim * c->kv_elt / 16;
    const unsigned groups = (unsigned)((pieces + 3) / 4);
    dynts::evict_compact_kernel<<<dim3(2 * groups, (unsigned)c->slabs(), 1), dynts::kCompactThreads, 0, c->stream>>>(p);
    CUDA_TRY(cudaGetLastError());
    c->launches += 2;
  }
  for (int b = 0; b < Nb; ++b)
    if (c->active_h[b]) c->len_h[b] = std::min(c->len_h[b], targets[b]);
  return DYNTS_OK;
}

}  // namespace

extern "C" {

const char* dynts_last_error(void) { return g_err; }
const char* dynts_version(void) { return "dynts-b200 0.1 (sm_100a)"; }

dynts_cache_t* dynts_cache_create(int layers, int kv_heads, int head_dim, int budget, int window) {
  dynts_cache* c = new (std::nothrow) dynts_cache();
  if (!c) {
    fail(DYNTS_ERR_OOM, "out of host memory");
    return nullptr;
  }
  memset(&c->cfg, 0, sizeof(c->cfg));
  c->cfg.layers = layers;
  c->cfg.batch = 1;
  c->cfg.q_heads = kv_heads;
  c->cfg.kv_heads = kv_heads;
  c->cfg.head_dim = head_dim;
  c->cfg.budget = budget;
  c->cfg.window = window;
  c->cfg.evict_interval = std::max(window, 64);
  c->cfg.dtype = DYNTS_BF16;
  if (!config_ok(&c->cfg, nullptr)) {
    fail(DYNTS_ERR_INVALID_ARG, "invalid arguments: layers %d kv_heads %d head_dim %d budget %d window %d", layers,
         kv_heads, head_dim, budget, window);
    delete c;
    return nullptr;
  }
  return c;
}

dynts_status_t dynts_cache_set_shape(dynts_cache_t* c, int batch, int q_heads, int dtype, int evict_interval) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (c->ready) return fail(DYNTS_ERR_STATE, "shape is fixed after the first prefill or decode");
  dynts_config_t t = c->cfg;
  t.batch = batch;
  t.q_heads = q_heads;
  t.dtype = dtype;
  t.evict_interval = evict_interval;
  if (!config_ok(&t, nullptr)) return fail(DYNTS_ERR_INVALID_ARG, "invalid shape");
  c->cfg = t;
  return DYNTS_OK;
}

size_t dynts_cache_bytes(const dynts_config_t* cfg) {
  int cap = 0;
  if (!config_ok(cfg, &cap)) return 0;
  return make_layout(cfg, cap).total;
}

dynts_status_t dynts_cache_create_ex(const dynts_config_t* cfg, dynts_cache_t** out) {
  if (!out) return fail(DYNTS_ERR_INVALID_ARG, "NULL out");
  *out = nullptr;
  if (!config_ok(cfg, nullptr)) return fail(DYNTS_ERR_INVALID_ARG, "invalid cache configuration");
  dynts_cache* c = new (std::nothrow) dynts_cache();
  if (!c) return fail(DYNTS_ERR_OOM, "out of host memory");
  c->cfg = *cfg;
  c->stream = static_cast<cudaStream_t>(cfg->stream);
  dynts_status_t st = materialise(c);
  if (st != DYNTS_OK) {
    if (c->owns_storage && c->base) cudaFree(c->base);
    if (c->err_host) cudaFreeHost(c->err_host);
    delete c;
    return st;
  }
  *out = c;
  return DYNTS_OK;
}

void dynts_cache_destroy(dynts_cache_t* c) {
  if (!c) return;
  if (c->ready) cudaStreamSynchronize(c->stream);
  if (c->owns_storage && c->base) cudaFree(c->base);
  if (c->stage_dev) cudaFree(c->stage_dev);
  if (c->err_host) cudaFreeHost(c->err_host);
  delete c;
}

dynts_status_t dynts_cache_set_stream(dynts_cache_t* c, void* stream) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (c->ready) {  // score passes still recorded are applied on the stream they belong to
    dynts_status_t fs_ = flush_pending(c);
    if (fs_ != DYNTS_OK) return fs_;
  }
  c->stream = static_cast<cudaStream_t>(stream);
  return DYNTS_OK;
}

dynts_status_t dynts_prefill(dynts_cache_t* c, const void* k, const void* v, int n_tokens, int n_pinned) {
  return do_prefill(c, -1, k, v, n_tokens, n_pinned);
}

}  // extern "C"

namespace {

dynts_status_t prompt_attn(dynts_cache* c, const void* q, const void* k, const void* v, void* out, int n_tokens, int n_layers) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (!q || !out || !k || !v || !aligned16(q) || !aligned16(out) || !aligned16(k) || !aligned16(v))
    return fail(DYNTS_ERR_INVALID_ARG, "q, k, v and out must be non-NULL and 16-byte aligned");
  if ((c->cfg.dtype != DYNTS_BF16 && c->cfg.dtype != DYNTS_BF16_KV8) || c->cfg.head_dim != 128)
    return fail(DYNTS_ERR_INVALID_ARG, "prefill attention needs bf16 q/k/v and head_dim 128");
  if (n_tokens < 1) return fail(DYNTS_ERR_INVALID_ARG, "n_tokens must be positive");
  dynts_status_t st = materialise(c);
  if (st != DYNTS_OK) return st;
  const long long lb = (long long)n_layers * c->cfg.batch;
  const long long n_qt = (n_tokens + dynts::kPfRows - 1) / dynts::kPfRows;
  if (lb * c->cfg.q_heads * n_qt >= (1ll << 30) || (long long)n_tokens * 256 >= (1ll << 40))
    return fail(DYNTS_ERR_INVALID_ARG, "layers x batch %lld with n_tokens %d beyond the launch limits", lb, n_tokens);
  if (!c->attr_prefill) {
    CUDA_TRY(cudaFuncSetAttribute(dynts::prefill_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, dynts::kPfSmemBytes));
    c->attr_prefill = true;
  }
  // Tensor maps over the caller's tensors, [heads][n_tokens][128]: a box never reaches into the next
  // head, rows beyond the prompt come back as zeros.  128-byte swizzle, boxes of 64 elements.
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
  if (!fn || qres != cudaDriverEntryPointSuccess) return fail(DYNTS_ERR_CUDA, "the driver has no cuTensorMapEncodeTiled");
  tensor_map_encode_fn encode = reinterpret_cast<tensor_map_encode_fn>(fn);
  CUtensorMap mq, mk, mv;
  const cuuint64_t strides[2] = {256, (cuuint64_t)n_tokens * 256};
  const cuuint32_t estr[3] = {1, 1, 1};
  auto make = [&](CUtensorMap* m, const void* base, int heads, int box_rows) -> CUresult {
    const cuuint64_t dims[3] = {128, (cuuint64_t)n_tokens, (cuuint64_t)lb * heads};
    const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    return encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  };
  CUresult r = make(&mq, q, c->cfg.q_heads, dynts::kPfRows);
  if (r == CUDA_SUCCESS) r = make(&mk, k, c->cfg.kv_heads, dynts::kPfKeys);
  if (r == CUDA_SUCCESS) r = make(&mv, v, c->cfg.kv_heads, dynts::kPfKeys);
  if (r != CUDA_SUCCESS) return fail(DYNTS_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
  dynts::PrefillAttnParams p;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.err = c->err_dev;
  p.stop = reinterpret_cast<int*>(c->ticket()) + 4;  // a spare word of the ticket block (zero since the cache was created)
  p.T = n_tokens;
  p.Hq = c->cfg.q_heads;
  p.Hkv = c->cfg.kv_heads;
  p.n_qt = (int)n_qt;
  p.n_heads = (int)(lb * c->cfg.q_heads);
  p.scale_log2 = (float)(1.4426950408889634 / std::sqrt(128.0));
  // two CTAs per SM (what their shared memory allows), each looping over its share of the (query tile, head) items
  const long long n_work = n_qt * p.n_heads;
  const unsigned grid = (unsigned)std::min<long long>(n_work, 2ll * c->sm_count);
  dynts::prefill_attn_kernel<<<grid, dynts::kPfThreads, dynts::kPfSmemBytes, c->stream>>>(p, mq, mk, mv);
  CUDA_TRY(cudaGetLastError());
  c->launches += 1;
  return DYNTS_OK;
}

}  // namespace

extern "C" {

dynts_status_t dynts_prompt_attn(dynts_cache_t* c, const void* q, const void* k, const void* v, void* out, int n_tokens) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  return prompt_attn(c, q, k, v, out, n_tokens, c->cfg.layers);
}

dynts_status_t dynts_prefill_attn_layer(dynts_cache_t* c, int layer, const void* q, const void* k, const void* v, void* out,
                                        int n_tokens, int n_pinned) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (layer < 0 || layer >= c->cfg.layers) return fail(DYNTS_ERR_INVALID_ARG, "layer %d out of range", layer);
  if (!q || !out || !aligned16(q) || !aligned16(out))
    return fail(DYNTS_ERR_INVALID_ARG, "q and out must be non-NULL and 16-byte aligned");
  if ((c->cfg.dtype != DYNTS_BF16 && c->cfg.dtype != DYNTS_BF16_KV8) || c->cfg.head_dim != 128)
    return fail(DYNTS_ERR_INVALID_ARG, "prefill attention needs bf16 q/k/v and head_dim 128");
  if (n_tokens < 1) return fail(DYNTS_ERR_INVALID_ARG, "n_tokens must be positive");
  dynts_status_t st = do_prefill(c, -1, k, v, n_tokens, n_pinned, layer);  // this layer's rows; lengths with the last layer
  if (st != DYNTS_OK) return st;
  return prompt_attn(c, q, k, v, out, n_tokens, 1);
}

dynts_status_t dynts_cache_refresh_lengths(dynts_cache_t* c) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (!c->ready) return DYNTS_OK;
  if (c->layer_cursor != 0) return fail(DYNTS_ERR_STATE, "a layer-by-layer step is in progress");
  CUDA_TRY(cudaStreamSynchronize(c->stream));
  const int Nb = c->cfg.batch;
  CUDA_TRY(cudaMemcpy(c->len_h.data(), c->len(), Nb * sizeof(int), cudaMemcpyDeviceToHost));
  CUDA_TRY(cudaMemcpy(c->tot_h.data(), c->tot(), Nb * sizeof(int), cudaMemcpyDeviceToHost));
  return DYNTS_OK;
}

dynts_status_t dynts_prefill_attn(dynts_cache_t* c, const void* q, const void* k, const void* v, void* out, int n_tokens,
                                  int n_pinned) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (!q || !out || !aligned16(q) || !aligned16(out))
    return fail(DYNTS_ERR_INVALID_ARG, "q and out must be non-NULL and 16-byte aligned");
  if ((c->cfg.dtype != DYNTS_BF16 && c->cfg.dtype != DYNTS_BF16_KV8) || c->cfg.head_dim != 128)
    return fail(DYNTS_ERR_INVALID_ARG, "prefill attention needs bf16 q/k/v and head_dim 128");
  if (n_tokens < 1) return fail(DYNTS_ERR_INVALID_ARG, "n_tokens must be positive");
  dynts_status_t st = do_prefill(c, -1, k, v, n_tokens, n_pinned);  // rows, positions, pins
  if (st != DYNTS_OK) return st;
  return dynts_prompt_attn(c, q, k, v, out, n_tokens);
}

dynts_status_t dynts_prefill_seq(dynts_cache_t* c, int seq, const void* k, const void* v, int n_tokens, int n_pinned) {
  if (seq < 0) return fail(DYNTS_ERR_INVALID_ARG, "sequence %d out of range", seq);
  return do_prefill(c, seq, k, v, n_tokens, n_pinned);
}

dynts_status_t dynts_decode_attn(dynts_cache_t* c, const void* q, const void* k_new, const void* v_new, void* out,
                                 float* scores) {
  dynts_status_t st = check_decode_args(c, q, k_new, v_new, out);
  if (st != DYNTS_OK) return st;
  st = materialise(c);
  if (st != DYNTS_OK) return st;
  if (c->layer_cursor != 0) return fail(DYNTS_ERR_STATE, "a layer-by-layer step is in progress");
  return launch_decode(c, 0, c->cfg.layers, q, k_new, v_new, out, scores, true);
}

dynts_status_t dynts_decode_attn_layer(dynts_cache_t* c, int layer, const void* q, const void* k_new,
                                       const void* v_new, void* out, float* scores) {
  dynts_status_t st = check_decode_args(c, q, k_new, v_new, out);
  if (st != DYNTS_OK) return st;
  st = materialise(c);
  if (st != DYNTS_OK) return st;
  if (layer != c->layer_cursor)
    return fail(DYNTS_ERR_STATE, "layer %d called, layer %d expected", layer, c->layer_cursor);
  const bool last = layer == c->cfg.layers - 1;
  st = launch_decode(c, layer, 1, q, k_new, v_new, out, scores, last);
  if (st == DYNTS_OK) c->layer_cursor = last ? 0 : layer + 1;
  return st;
}

dynts_status_t dynts_decode_attn_host(dynts_cache_t* c, const void* q, const void* k_new, const void* v_new,
                                      void* out) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (!q || !k_new || !v_new || !out) return fail(DYNTS_ERR_INVALID_ARG, "NULL tensor pointer");
  dynts_status_t st = materialise(c);
  if (st != DYNTS_OK) return st;
  if (c->layer_cursor != 0) return fail(DYNTS_ERR_STATE, "a layer-by-layer step is in progress");
  for (int b = 0; b < c->cfg.batch; ++b)
    if (c->active_h[b] && c->len_h[b] + 1 > c->cap)
      return fail(DYNTS_ERR_CAPACITY, "sequence %d is at capacity %d: evict before the next decode step", b, c->cap);
  const dynts_config_t& f = c->cfg;
  const size_t qb = align_up((size_t)f.layers * f.batch * f.q_heads * f.head_dim * c->elt, 256);
  const size_t kb = align_up((size_t)f.layers * f.batch * f.kv_heads * f.head_dim * c->elt, 256);
  const size_t need = 2 * qb + 2 * kb;
  if (c->stage_bytes < need) {
    if (c->stage_dev) cudaFree(c->stage_dev);
    c->stage_dev = nullptr;
    c->stage_bytes = 0;
    void* ptr = nullptr;
    cudaError_t e = cudaMalloc(&ptr, need);
    if (e != cudaSuccess) return fail(DYNTS_ERR_OOM, "cudaMalloc(%zu): %s", need, cudaGetErrorString(e));
    c->stage_dev = static_cast<char*>(ptr);
    c->stage_bytes = need;
  }
  char* dq = c->stage_dev;
  char* dk = dq + qb;
  char* dv = dk + kb;
  char* dout = dv + kb;
  const size_t qn = (size_t)f.layers * f.batch * f.q_heads * f.head_dim * c->elt;
  const size_t kn = (size_t)f.layers * f.batch * f.kv_heads * f.head_dim * c->elt;
  // Pinned, mapped host buffers (cudaHostAlloc / cudaHostRegister; what PyTorch's pin_memory gives)
  // are read by the kernel in place: each input element is read exactly once, so a staging copy
  // would only add three transfers' latency.  Other host memory is staged.
  auto device_view = [](const void* h) -> const void* {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, h) != cudaSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    if (a.type != cudaMemoryTypeHost || !a.devicePointer || !aligned16(a.devicePointer)) return nullptr;
    return a.devicePointer;
  };
  const void* vq = device_view(q);
  const void* vk = device_view(k_new);
  const void* vv = device_view(v_new);
  void* vo = const_cast<void*>(device_view(out));
  if (vq && vk && vv && vo) {  // the output rows are written to the host buffer by the kernel as well
    st = launch_decode(c, 0, f.layers, vq, vk, vv, vo, nullptr, true);
    if (st != DYNTS_OK) return st;
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    return DYNTS_OK;
  } else if (vq && vk && vv) {
    st = launch_decode(c, 0, f.layers, vq, vk, vv, dout, nullptr, true);
  } else {
    CUDA_TRY(cudaMemcpyAsync(dq, q, qn, cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(cudaMemcpyAsync(dk, k_new, kn, cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(cudaMemcpyAsync(dv, v_new, kn, cudaMemcpyHostToDevice, c->stream));
    st = launch_decode(c, 0, f.layers, dq, dk, dv, dout, nullptr, true);
  }
  if (st != DYNTS_OK) return st;
  CUDA_TRY(cudaMemcpyAsync(out, dout, qn, cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(cudaStreamSynchronize(c->stream));
  return DYNTS_OK;
}

dynts_status_t dynts_evict(dynts_cache_t* c, int budget) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (!c->ready) return fail(DYNTS_ERR_STATE, "cache holds nothing yet");
  if (c->layer_cursor != 0) return fail(DYNTS_ERR_STATE, "evict in the middle of a layer-by-layer step");
  std::vector<int> t(c->cfg.batch);
  for (int b = 0; b < c->cfg.batch; ++b) t[b] = budget > 0 ? budget : c->seq_budget[b];
  return do_evict(c, t.data());
}

dynts_status_t dynts_evict_global(dynts_cache_t* c, int budget) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (!c->ready) return fail(DYNTS_ERR_STATE, "cache holds nothing yet");
  if (c->layer_cursor != 0) return fail(DYNTS_ERR_STATE, "evict in the middle of a layer-by-layer step");
  std::vector<int> t(c->cfg.batch);
  for (int b = 0; b < c->cfg.batch; ++b) t[b] = budget > 0 ? budget : c->seq_budget[b];
  return do_evict(c, t.data(), true);
}

dynts_status_t dynts_aggregate_scores(dynts_cache_t* c, float* agg) {
  if (!c || !agg) return fail(DYNTS_ERR_INVALID_ARG, "NULL argument");
  if (!c->ready) return fail(DYNTS_ERR_STATE, "cache holds nothing yet");
  if (c->layer_cursor != 0) return fail(DYNTS_ERR_STATE, "a layer-by-layer step is in progress");
  {
    dynts_status_t fs_ = flush_pending(c);
    if (fs_ != DYNTS_OK) return fs_;
  }
  dynts::aggregate_scores_kernel<<<dim3((unsigned)((c->cap + 255) / 256), (unsigned)c->cfg.batch, 1), 256, 0, c->stream>>>(
      c->score(), agg, c->len(), c->active(), c->cfg.layers, c->cfg.batch, c->cfg.kv_heads, c->cap);
  CUDA_TRY(cudaGetLastError());
  c->launches += 1;
  return DYNTS_OK;
}

dynts_status_t dynts_evict_ex(dynts_cache_t* c, const int* seq_targets) {
  if (!c || !seq_targets) return fail(DYNTS_ERR_INVALID_ARG, "NULL argument");
  if (!c->ready) return fail(DYNTS_ERR_STATE, "cache holds nothing yet");
  if (c->layer_cursor != 0) return fail(DYNTS_ERR_STATE, "evict in the middle of a layer-by-layer step");
  for (int b = 0; b < c->cfg.batch; ++b)
    if (seq_targets[b] < 1) return fail(DYNTS_ERR_INVALID_ARG, "target of sequence %d must be positive", b);
  return do_evict(c, seq_targets);
}

dynts_status_t dynts_seq_reset(dynts_cache_t* c, int seq) {
  if (!c || seq < 0 || seq >= c->cfg.batch) return fail(DYNTS_ERR_INVALID_ARG, "bad cache or sequence");
  if (!c->ready) return fail(DYNTS_ERR_STATE, "cache holds nothing yet");
  if (c->layer_cursor != 0) return fail(DYNTS_ERR_STATE, "reset in the middle of a layer-by-layer step");
  {
    dynts_status_t fs_ = flush_pending(c);
    if (fs_ != DYNTS_OK) return fs_;
  }
  CUDA_TRY(cudaMemsetAsync(c->len() + seq, 0, sizeof(int), c->stream));
  CUDA_TRY(cudaMemsetAsync(c->tot() + seq, 0, sizeof(int), c->stream));
  CUDA_TRY(cudaMemsetAsync(c->pinned() + seq, 0, sizeof(int), c->stream));
  CUDA_TRY(cudaMemsetAsync(c->active() + seq, 0, sizeof(int), c->stream));
  c->len_h[seq] = 0;
  c->tot_h[seq] = 0;
  c->pinned_h[seq] = 0;
  c->active_h[seq] = 0;
  return DYNTS_OK;
}

int dynts_cache_len(const dynts_cache_t* c, int seq) {
  if (!c || seq < 0 || seq >= c->cfg.batch) return -1;
  if (!c->ready) return 0;
  return c->len_h[seq];
}

int dynts_cache_capacity(const dynts_cache_t* c) {
  if (!c) return -1;
  if (c->ready) return c->cap;
  int cap = 0;
  return config_ok(&c->cfg, &cap) ? cap : -1;
}

float* dynts_cache_scores(dynts_cache_t* c) {
  if (!c || !c->ready) return nullptr;
  if (flush_pending(c) != DYNTS_OK) return nullptr;  // score passes still recorded are applied on the stream first
  return c->score();
}

dynts_status_t dynts_cache_export(dynts_cache_t* c, int layer, int seq, int head, void* K, void* V, int* pos,
                                  float* score, int* n) {
  if (!c || !c->ready) return fail(DYNTS_ERR_STATE, "cache holds nothing yet");
  if (layer < 0 || layer >= c->cfg.layers || seq < 0 || seq >= c->cfg.batch || head < 0 || head >= c->cfg.kv_heads)
    return fail(DYNTS_ERR_INVALID_ARG, "slab index out of range");
  {
    dynts_status_t fs_ = flush_pending(c);
    if (fs_ != DYNTS_OK) return fs_;
  }
  CUDA_TRY(cudaStreamSynchronize(c->stream));
  const size_t slab = ((size_t)layer * c->cfg.batch + seq) * c->cfg.kv_heads + head;
  const int rows = c->len_h[seq];
  const size_t row_bytes = (size_t)c->cfg.head_dim * c->kv_elt;
  if (K) CUDA_TRY(cudaMemcpy(K, static_cast<char*>(c->K()) + slab * c->cap * row_bytes, rows * row_bytes, cudaMemcpyDeviceToHost));
  if (V) CUDA_TRY(cudaMemcpy(V, static_cast<char*>(c->V()) + slab * c->cap * row_bytes, rows * row_bytes, cudaMemcpyDeviceToHost));
  if (pos) CUDA_TRY(cudaMemcpy(pos, c->pos() + slab * c->cap, rows * sizeof(int), cudaMemcpyDeviceToHost));
  if (score) CUDA_TRY(cudaMemcpy(score, c->score() + slab * c->cap, rows * sizeof(float), cudaMemcpyDeviceToHost));
  if (n) *n = rows;
  return DYNTS_OK;
}

dynts_status_t dynts_cache_import(dynts_cache_t* c, int layer, int seq, int head, const void* K, const void* V,
                                  const int* pos, const float* score, int n, int n_pinned) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  dynts_status_t st = materialise(c);
  if (st != DYNTS_OK) return st;
  if (layer < 0 || layer >= c->cfg.layers || seq < 0 || seq >= c->cfg.batch || head < 0 || head >= c->cfg.kv_heads)
    return fail(DYNTS_ERR_INVALID_ARG, "slab index out of range");
  if (!K || !V || !pos || !score) return fail(DYNTS_ERR_INVALID_ARG, "NULL buffer");
  if (n < 0 || n > c->cap) return fail(DYNTS_ERR_CAPACITY, "%d rows exceed capacity %d", n, c->cap);
  if (n_pinned < 0 || n_pinned > n) return fail(DYNTS_ERR_INVALID_ARG, "n_pinned out of range");
  if (c->layer_cursor != 0) return fail(DYNTS_ERR_STATE, "import in the middle of a layer-by-layer step");
  {
    dynts_status_t fs_ = flush_pending(c);
    if (fs_ != DYNTS_OK) return fs_;
  }
  CUDA_TRY(cudaStreamSynchronize(c->stream));
  const size_t slab = ((size_t)layer * c->cfg.batch + seq) * c->cfg.kv_heads + head;
  const size_t row_bytes = (size_t)c->cfg.head_dim * c->kv_elt;
  CUDA_TRY(cudaMemcpy(static_cast<char*>(c->K()) + slab * c->cap * row_bytes, K, n * row_bytes, cudaMemcpyHostToDevice));
  CUDA_TRY(cudaMemcpy(static_cast<char*>(c->V()) + slab * c->cap * row_bytes, V, n * row_bytes, cudaMemcpyHostToDevice));
  CUDA_TRY(cudaMemcpy(c->pos() + slab * c->cap, pos, n * sizeof(int), cudaMemcpyHostToDevice));
  CUDA_TRY(cudaMemcpy(c->score() + slab * c->cap, score, n * sizeof(float), cudaMemcpyHostToDevice));
  CUDA_TRY(cudaMemset(c->comp() + slab * c->cap, 0, n * sizeof(float)));
  int next = n > 0 ? pos[n - 1] + 1 : 0;
  int one = 1;
  CUDA_TRY(cudaMemcpy(c->len() + seq, &n, sizeof(int), cudaMemcpyHostToDevice));
  CUDA_TRY(cudaMemcpy(c->tot() + seq, &next, sizeof(int), cudaMemcpyHostToDevice));
  CUDA_TRY(cudaMemcpy(c->pinned() + seq, &n_pinned, sizeof(int), cudaMemcpyHostToDevice));
  CUDA_TRY(cudaMemcpy(c->active() + seq, &one, sizeof(int), cudaMemcpyHostToDevice));
  c->len_h[seq] = n;
  c->tot_h[seq] = next;
  c->pinned_h[seq] = n_pinned;
  c->active_h[seq] = 1;
  return DYNTS_OK;
}

dynts_status_t dynts_poll_error(dynts_cache_t* c) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (c->err_host && *reinterpret_cast<volatile int*>(c->err_host) != 0) {
    const int word = *reinterpret_cast<volatile int*>(c->err_host);
    int dbg[24] = {0};
    if (c->ready && (word & dynts::kErrStreamBounds))
      cudaMemcpy(dbg, reinterpret_cast<int*>(c->ticket()) + 8, sizeof(dbg), cudaMemcpyDeviceToHost);
    return fail(DYNTS_ERR_DEVICE,
                "device status word 0x%x (producer: layer %d seq %d head %d chunk %d len %d item %d cta %d smem 0x%x; "
                "consumer: layer %d seq %d head %d chunk %d n %d item %d cta %d seg %d; sharers %d..%d cta %d first chunk %d)",
                word, dbg[0], dbg[1], dbg[2], dbg[3], dbg[4], dbg[5], dbg[6], dbg[7], dbg[8], dbg[9], dbg[10], dbg[11],
                dbg[12], dbg[13], dbg[14], dbg[15], dbg[16], dbg[17], dbg[18], dbg[19]);
  }
  return DYNTS_OK;
}

dynts_status_t dynts_synchronize(dynts_cache_t* c) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  {
    dynts_status_t fs_ = flush_pending(c);
    if (fs_ != DYNTS_OK) return fs_;
  }
  CUDA_TRY(cudaStreamSynchronize(c->stream));
  return DYNTS_OK;
}

dynts_status_t dynts_cache_set_launch(dynts_cache_t* c, int cluster, int variant) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (!(cluster == 0 || cluster == 1 || cluster == 2 || cluster == 4 || cluster == 8 || cluster == 16))
    return fail(DYNTS_ERR_INVALID_ARG, "cluster size must be 0, 1, 2, 4, 8 or 16");
  if (variant < 0 || variant > 3) return fail(DYNTS_ERR_INVALID_ARG, "variant must be 0, 1, 2 or 3");
  c->cluster = cluster;
  c->variant = variant;
  return DYNTS_OK;
}

dynts_status_t dynts_cache_set_wait_limit(dynts_cache_t* c, unsigned int polls) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (polls < 64u) return fail(DYNTS_ERR_INVALID_ARG, "the limit must be at least 64 polls");
  c->wait_limit = polls;
  return DYNTS_OK;
}

dynts_status_t dynts_debug_drop_tile_load(dynts_cache_t* c, int item) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (item < 0) return fail(DYNTS_ERR_INVALID_ARG, "item must not be negative");
  c->drop_item = item;
  return DYNTS_OK;
}

dynts_status_t dynts_cache_set_evict_launch(dynts_cache_t* c, int split) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (!(split == -1 || split == 0 || split == 1 || split == 2 || split == 4 || split == 8))
    return fail(DYNTS_ERR_INVALID_ARG, "split must be -1, 0, 1, 2, 4 or 8");
  c->evict_split = split;
  return DYNTS_OK;
}

long long dynts_cache_launch_count(const dynts_cache_t* c) { return c ? c->launches : -1; }

dynts_status_t dynts_cache_set_score_source(dynts_cache_t* c, int source) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (source != DYNTS_SCORE_ATTENTION && source != DYNTS_SCORE_EXTERNAL)
    return fail(DYNTS_ERR_INVALID_ARG, "score source must be DYNTS_SCORE_ATTENTION or DYNTS_SCORE_EXTERNAL");
  if (c->layer_cursor != 0) return fail(DYNTS_ERR_STATE, "a layer-by-layer step is in progress");
  {
    dynts_status_t fs_ = flush_pending(c);
    if (fs_ != DYNTS_OK) return fs_;
  }
  c->score_source = source;
  return DYNTS_OK;
}

dynts_status_t dynts_cache_set_kv_scale(dynts_cache_t* c, float k_scale, float v_scale) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (c->cfg.dtype != DYNTS_BF16_KV8) return fail(DYNTS_ERR_INVALID_ARG, "the cache does not hold 8-bit rows");
  if (!(k_scale > 0.f) || !(v_scale > 0.f) || std::isinf(k_scale) || std::isinf(v_scale))
    return fail(DYNTS_ERR_INVALID_ARG, "scales must be positive and finite (%g, %g)", (double)k_scale, (double)v_scale);
  if (c->ready)
    for (int b = 0; b < c->cfg.batch; ++b)
      if (c->len_h[b] > 0) return fail(DYNTS_ERR_STATE, "rows are already stored with the current scales");
  c->k_scale = k_scale;
  c->v_scale = v_scale;
  return DYNTS_OK;
}

dynts_status_t dynts_append_scores(dynts_cache_t* c, const float* s_new) {
  if (!c || !s_new) return fail(DYNTS_ERR_INVALID_ARG, "NULL argument");
  if (!c->ready) return fail(DYNTS_ERR_STATE, "cache holds nothing yet");
  if (c->layer_cursor != 0) return fail(DYNTS_ERR_STATE, "a layer-by-layer step is in progress");
  {
    dynts_status_t fs_ = flush_pending(c);
    if (fs_ != DYNTS_OK) return fs_;
  }
  const int n_slabs = (int)c->slabs();
  dynts::append_scores_kernel<<<(n_slabs + 255) / 256, 256, 0, c->stream>>>(c->score(), c->comp(), c->len(), c->active(), s_new,
                                                                          n_slabs, c->cfg.batch, c->cfg.kv_heads, c->cap);
  CUDA_TRY(cudaGetLastError());
  c->launches += 1;
  return DYNTS_OK;
}

dynts_status_t dynts_evict_at_budget(dynts_cache_t* c, int budget_B, double ratio) {
  if (!c) return fail(DYNTS_ERR_INVALID_ARG, "NULL cache");
  if (!c->ready) return fail(DYNTS_ERR_STATE, "cache holds nothing yet");
  if (c->layer_cursor != 0) return fail(DYNTS_ERR_STATE, "evict in the middle of a layer-by-layer step");
  if (budget_B < 1 || budget_B > c->cap || !(ratio >= 0.0 && ratio <= 1.0))
    return fail(DYNTS_ERR_INVALID_ARG, "budget %d outside [1, capacity %d] or ratio %g outside [0, 1]", budget_B, c->cap, ratio);
  const int Nb = c->cfg.batch;
  std::vector<int> t(Nb);
  for (int b = 0; b < Nb; ++b) {
    t[b] = c->cap;  // no eviction for this sequence
    if (!c->active_h[b] || c->len_h[b] < budget_B) continue;
    const int w_s = budget_B - c->pinned_h[b] - c->cfg.window;
    if (w_s < 0)
      return fail(DYNTS_ERR_BUDGET, "sequence %d: question window %d + local window %d exceed the budget %d", b,
                  c->pinned_h[b], c->cfg.window, budget_B);
    t[b] = c->pinned_h[b] + (int)std::floor(ratio * (double)w_s) + c->cfg.window;
  }
  return do_evict(c, t.data());
}

dynts_status_t dynts_evict_stats(dynts_cache_t* c, long long* rows_scanned, long long* rows_moved) {
  if (!c || !c->ready) return fail(DYNTS_ERR_STATE, "cache holds nothing yet");
  CUDA_TRY(cudaStreamSynchronize(c->stream));
  std::vector<int> h(c->slabs() * 4);
  CUDA_TRY(cudaMemcpy(h.data(), c->hdr(), h.size() * sizeof(int), cudaMemcpyDeviceToHost));
  long long scanned = 0, moved = 0;
  for (size_t s = 0; s < c->slabs(); ++s) {
    const int first = h[4 * s], kept = h[4 * s + 1], old_len = h[4 * s + 2];
    if (old_len > kept) {  // this slab was evicted by the last eviction
      scanned += old_len;
      moved += kept > first ? kept - first : 0;
    }
  }
  if (rows_scanned) *rows_scanned = scanned;
  if (rows_moved) *rows_moved = moved;
  return DYNTS_OK;
}

/* ---- Importance Predictor head ------------------------------------------------------------ */

}  // extern "C"

namespace {

// K-slices of a layer with `rows` outputs and K inputs: enough CTAs to fill the GPU (about 256),
// slices that are multiples of 256 elements and fit shared memory (bf16 hi and lo halves of a tile of 16
// sequences, several CTAs per SM).
int mlp_k_slices(int rows, int K) {
  const int units = K / 256;
  const int row_blocks = (rows + dynts::kMlpRowsPerCta - 1) / dynts::kMlpRowsPerCta;
  int best = units;  // finest split as a fallback
  for (int ks = 1; ks <= units; ++ks) {
    if (units % ks) continue;
    if ((size_t)(K / ks + dynts::kMlpPad) * dynts::kMlpBatchTile * 4 > 72 * 1024) continue;
    if (row_blocks * ks >= 256) return ks;
    best = ks;
  }
  return best;
}

bool g_mlp_attr[64] = {false};  // per device: function attributes are set once per device

}  // namespace

extern "C" {

size_t dynts_predictor_mlp_scratch_bytes(int d, int batch) {
  if (d < 512 || d % 512 || batch < 1) return 0;
  const size_t p1 = (size_t)mlp_k_slices(2 * d, d) * batch * (2 * d);
  const size_t p2 = (size_t)mlp_k_slices(d / 2, 2 * d) * batch * (d / 2);
  return (p1 + p2) * sizeof(float);
}

dynts_status_t dynts_predictor_mlp(const void* h, const void* W1, const float* b1, const void* W2, const float* b2,
                                   const void* W3, const float* b3, int d, int batch, int activation, void* scratch,
                                   size_t scratch_bytes, float* scores, void* stream) {
  if (!h || !W1 || !W2 || !W3 || !scratch || !scores) return fail(DYNTS_ERR_INVALID_ARG, "NULL tensor pointer");
  if (!aligned16(h) || !aligned16(W1) || !aligned16(W2) || !aligned16(W3) || !aligned16(scratch))
    return fail(DYNTS_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned");
  if (d < 512 || d % 512 || batch < 1) return fail(DYNTS_ERR_INVALID_ARG, "d must be a multiple of 512, batch >= 1");
  if (activation != 0 && activation != 1) return fail(DYNTS_ERR_INVALID_ARG, "activation must be 0 (none) or 1 (ReLU)");
  const size_t need = dynts_predictor_mlp_scratch_bytes(d, batch);
  if (scratch_bytes < need) return fail(DYNTS_ERR_OOM, "scratch too small: %zu < %zu bytes", scratch_bytes, need);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int dev = 0;
  CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return fail(DYNTS_ERR_INVALID_ARG, "device index %d not supported", dev);
  if (!g_mlp_attr[dev]) {
    CUDA_TRY(cudaFuncSetAttribute(dynts::mlp_layer_kernel<1, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024));
    CUDA_TRY(cudaFuncSetAttribute(dynts::mlp_layer_kernel<2, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024));
    g_mlp_attr[dev] = true;
  }
  const int NT = batch > 8 ? 16 : 8;  // sequences per batch tile
  const int ks1 = mlp_k_slices(2 * d, d), ks2 = mlp_k_slices(d / 2, 2 * d);
  float* parts1 = static_cast<float*>(scratch);
  float* parts2 = parts1 + (size_t)ks1 * batch * (2 * d);
  const unsigned tiles = (unsigned)((batch + NT - 1) / NT);

  dynts::MlpLayerParams p;
  p.W = static_cast<const __nv_bfloat16*>(W1);
  p.xh = static_cast<const __nv_bfloat16*>(h);
  p.xparts = nullptr;
  p.xbias = nullptr;
  p.yparts = parts1;
  p.rows = 2 * d;
  p.K = d;
  p.Nb = batch;
  p.n_parts = 0;
  p.act = 0;
  p.k_slice = d / ks1;
  // For batch tiles of 16 sequences, up to 8 K slices (a power of two) form a cluster that finishes
  // the layer's values itself; with tiles of 8 the consumers' re-reduction of the partial sums is
  // cheap (a few KB per CTA) and the cluster barriers cost more than they save (25.2 vs 23.3 us at
  // batch 1; 64 vs 42 us the other way at batch 16).
  auto clustered = [NT](int ks) { return NT == 16 && ks <= 8 && (ks & (ks - 1)) == 0; };
  p.cluster_reduce = clustered(ks1) ? 1 : 0;
  p.ybias = b1;
  p.yact = activation;
  auto launch_layer = [&](const dynts::MlpLayerParams& q, int ks) -> cudaError_t {
    // hi halves of the staged input, and lo halves when the input is fp32
    const size_t smem = (size_t)(q.xh ? 1 : 2) * NT * (q.k_slice + dynts::kMlpPad) * 2;
    // Four warps of 16 weight rows per CTA.  (Measured at d = 4096, batch 1: CTAs of one, two and
    // eight warps took 45, 27 and 23.7 us per call against 23.3 us.)
    constexpr int warps = dynts::kMlpWarps;
    const dim3 grid(tiles, (unsigned)((q.rows + 16 * warps - 1) / (16 * warps)), (unsigned)ks);
    cudaLaunchConfig_t lc;
    memset(&lc, 0, sizeof(lc));
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see griddepcontrol.wait in the kernel
    at[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at;
    lc.numAttrs = 1;
    if (q.cluster_reduce && ks > 1) {
      at[1].id = cudaLaunchAttributeClusterDimension;
      at[1].val.clusterDim.x = 1;
      at[1].val.clusterDim.y = 1;
      at[1].val.clusterDim.z = (unsigned)ks;
      lc.numAttrs = 2;
    }
    lc.stream = st;
    lc.gridDim = grid;
    lc.blockDim = dim3((unsigned)warps * 32, 1, 1);
    lc.dynamicSmemBytes = smem;
    if (NT == 16) return cudaLaunchKernelEx(&lc, dynts::mlp_layer_kernel<2, 4>, q);
    return cudaLaunchKernelEx(&lc, dynts::mlp_layer_kernel<1, 4>, q);
  };
  CUDA_TRY(launch_layer(p, ks1));

  const bool done1 = p.cluster_reduce != 0;  // layer 1's values are finished (bias and activation applied)
  p.W = static_cast<const __nv_bfloat16*>(W2);
  p.xh = nullptr;
  p.xparts = parts1;
  p.xbias = done1 ? nullptr : b1;
  p.yparts = parts2;
  p.rows = d / 2;
  p.K = 2 * d;
  p.n_parts = done1 ? 1 : ks1;
  p.act = done1 ? 0 : activation;
  p.k_slice = 2 * d / ks2;
  p.cluster_reduce = clustered(ks2) ? 1 : 0;
  p.ybias = b2;
  p.yact = activation;
  CUDA_TRY(launch_layer(p, ks2));
  const bool done2 = p.cluster_reduce != 0;

  {
    cudaLaunchConfig_t lc;
    memset(&lc, 0, sizeof(lc));
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at;
    lc.numAttrs = 1;
    lc.stream = st;
    lc.gridDim = dim3((unsigned)batch, 1, 1);
    lc.blockDim = dim3(dynts::kMlpHeadThreads, 1, 1);
    CUDA_TRY(cudaLaunchKernelEx(&lc, dynts::mlp_head_kernel, static_cast<const __nv_bfloat16*>(W3), (const float*)parts2,
                                done2 ? (const float*)nullptr : b2, b3, scores, d / 2, batch, done2 ? 1 : ks2,
                                done2 ? 0 : activation));
  }
  return DYNTS_OK;
}

/* ---- eviction for callers that cannot allocate -------------------------------------------- */

}  // extern "C" (the scratch array and its helpers have internal linkage)

namespace {

// Scratch of dynts_evict_noalloc: a small header (length, pinned, target, status), then the
// per-slab headers, then the gather lists.  Every GPU that loads this library holds these
// 4 MiB until the process exits.
constexpr size_t kNoAllocInts = (size_t)1 << 20;
constexpr size_t kNoAllocHeaderInts = 64;
static __device__ __align__(256) int g_noalloc_scratch[kNoAllocInts];

constexpr int kMaxDevices = 64;
int* g_noalloc_ptr[kMaxDevices] = {nullptr};
std::mutex g_noalloc_mutex;

__global__ void noalloc_setup_kernel(int* hdr, int n_rows, int n_pinned, int target) {
  hdr[0] = n_rows;    // plays the role of the per-sequence length array (one sequence)
  hdr[1] = n_pinned;
  hdr[2] = target;
  hdr[3] = 0;         // status word
}

}  // namespace

extern "C" {

dynts_status_t dynts_evict_noalloc(void* K, void* V, int* pos, float* score, int n_slabs, int head_dim, int dtype,
                                   int capacity, int n_rows, int n_pinned, int window, int target, void* stream) {
  if (!K || !V || !pos || !score) return fail(DYNTS_ERR_INVALID_ARG, "NULL tensor pointer");
  if (!aligned16(K) || !aligned16(V)) return fail(DYNTS_ERR_INVALID_ARG, "K and V must be 16-byte aligned");
  if (dtype != DYNTS_BF16 && dtype != DYNTS_FP32 && dtype != DYNTS_BF16_KV8)
    return fail(DYNTS_ERR_INVALID_ARG, "unknown dtype %d", dtype);
  if (n_slabs < 1 || head_dim < 8 || head_dim % 8 || head_dim > 256 || capacity < 1 ||
      (dtype == DYNTS_BF16_KV8 && head_dim % 16))
    return fail(DYNTS_ERR_INVALID_ARG, "bad shape: n_slabs %d head_dim %d capacity %d", n_slabs, head_dim, capacity);
  if (n_rows < 0 || n_rows > capacity || n_pinned < 0 || n_pinned > n_rows || window < 0 || target < 1)
    return fail(DYNTS_ERR_INVALID_ARG, "bad lengths: n_rows %d n_pinned %d window %d target %d", n_rows, n_pinned,
                window, target);
  const size_t hdr_ints = align_up((size_t)n_slabs * 4, 64);
  const size_t need = kNoAllocHeaderInts + hdr_ints + (size_t)n_slabs * capacity;
  if (need > kNoAllocInts)
    return fail(DYNTS_ERR_CAPACITY,
                "n_slabs * capacity = %zu rows need %zu scratch ints; the built-in scratch holds %zu (about %zu rows)",
                (size_t)n_slabs * capacity, need, kNoAllocInts, kNoAllocInts - kNoAllocHeaderInts - hdr_ints);
  if ((size_t)capacity * 8 > 200 * 1024)
    return fail(DYNTS_ERR_CAPACITY, "capacity %d exceeds the selection kernel's shared memory", capacity);
  if (n_rows <= target) return DYNTS_OK;  // nothing to evict
  if (n_pinned + window > target)
    return fail(DYNTS_ERR_BUDGET, "question window %d + local window %d exceed target %d", n_pinned, window, target);

  int dev = -1;
  CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return fail(DYNTS_ERR_INVALID_ARG, "device index %d not supported", dev);
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);  // the scratch is shared: one call at a time
  if (!g_noalloc_ptr[dev]) {
    // Once per device, with that device current: the array's name is only a host-side stand-in,
    // the kernels need its device address.
    int* ptr = nullptr;
    CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_scratch));
    CUDA_TRY(cudaFuncSetAttribute(dynts::evict_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    g_noalloc_ptr[dev] = ptr;
  }
  int* base = g_noalloc_ptr[dev];
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  dynts::EvictParams p;
  p.K = K;
  p.V = V;
  p.pos = pos;
  p.score = score;
  p.comp = nullptr;
  p.key = nullptr;
  p.len = base + 0;
  p.pinned = base + 1;
  p.target = base + 2;
  p.err = base + 3;
  p.hdr = base + kNoAllocHeaderInts;
  p.src = base + kNoAllocHeaderInts + hdr_ints;
  p.L = 1;
  p.Nb = 1;
  p.Hkv = n_slabs;
  p.d = head_dim;
  p.cap = capacity;
  p.window = window;
  p.elt_bytes = kv_elt_bytes_of(dtype);
  noalloc_setup_kernel<<<1, 1, 0, st>>>(base, n_rows, n_pinned, target);
  CUDA_TRY(cudaGetLastError());
  dynts::evict_select_kernel<<<(unsigned)n_slabs, dynts::kSelectThreads, (size_t)capacity * 8, st>>>(p);
  CUDA_TRY(cudaGetLastError());
  const int pieces = head_dim * p.elt_bytes / 16;
  const unsigned groups = (unsigned)((pieces + 3) / 4);
  dynts::evict_compact_kernel<<<dim3(2 * groups, (unsigned)n_slabs, 1), dynts::kCompactThreads, 0, st>>>(p);
  CUDA_TRY(cudaGetLastError());
  return DYNTS_OK;
}

dynts_status_t dynts_evict_noalloc_status(void* stream) {
  int dev = -1;
  CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return fail(DYNTS_ERR_INVALID_ARG, "device index %d not supported", dev);
  int* base = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    base = g_noalloc_ptr[dev];
  }
  if (!base) return DYNTS_OK;  // no call on this device yet
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int word = 0;  // (a pageable destination: the copy is staged by the runtime, nothing is allocated here)
  CUDA_TRY(cudaMemcpyAsync(&word, base + 3, sizeof(int), cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaStreamSynchronize(st));
  if (word != 0) return fail(DYNTS_ERR_DEVICE, "the last dynts_evict_noalloc call found inconsistent lengths on the device (status word 0x%x) and moved nothing for those slabs", word);
  return DYNTS_OK;
}

}  // extern "C"

