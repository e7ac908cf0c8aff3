// C ABI of libsds (see include/sds.h): context, workspace carving, call-order checks and the
// host loop of sds_sample_all. All device work is in the kernels this file launches.
#include "../../include/sds.h"

#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "sds_device.cuh"
#include "sds_internal.h"
#include "sds_tc.h"

using namespace sds;

namespace {

enum State { kCreated = 0, kBound, kReady, kDrafted, kVerified };

constexpr size_t kAlign = 256;
constexpr size_t kNone = (size_t)-1;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Carve {
  size_t off = 0;
  size_t take(size_t bytes) {
    const size_t o = off;
    off = align_up(off + bytes);
    return o;
  }
};

// byte offsets of every workspace region
struct Layout {
  size_t a, c, sigma, tcond;
  size_t Y, Dc, T, X, Dq, Xb;
  size_t n, act, rowoff, rowk, ctl;
  size_t S1, S2, ell, logU, accmask, jstar, nfe_calls, nfe_rows;
  size_t rem;             // staged windows: positions left in a chain's window
  size_t Gk;
  size_t Gx, Gb, Pb, Dp;  // independent drafter: gathered rows (f32, bf16), its outputs per call and per row
  size_t ce;              // (C_k, E_k) of the target mixture as floats, for rows kept raw
  size_t adet, cdet;      // Picard drafter: deterministic sampler coefficients (Dp then holds draft means)
  size_t total;
};

// workspace regions private to one denoiser (the target, or the independent draft model)
struct DenLayout {
  size_t tcond, musq;
  size_t H0, H1;          // MLP hidden activations (bf16)
  size_t logits, R, Mt;   // large mixture: logits (f32), responsibilities (bf16), transposed means (bf16)
  size_t Xs, Ms;          // float mixture on tensor cores: 3 bf16 planes of the rows / of the means
  size_t flags;           // one int per 128 rows: responsibilities with a non-zero second or third plane
  size_t amax, hot;       // component of every one-hot row (-1: not one-hot); one int per 256 rows: some row not one-hot
  size_t xb;              // where a bf16 copy of this denoiser's input rows goes when the caller has none
};

struct Engine {
  sds_denoiser den{};
  std::vector<int32_t> mlp_dims;                 // copies of the caller's MLP description
  std::vector<const void*> mlp_W, mlp_temb;
  std::vector<const float*> mlp_bias;
  std::vector<double> tcond;
  DenLayout lay{};
  int64_t cap_rows = 0;                          // rows of the buffers this denoiser's GEMMs read
  bool musq_ready = false;
};

}  // namespace

struct sds_ctx {
  int64_t B = 0;
  int32_t d = 0, L = 0, K = 0;
  std::vector<float> a, c, sigma;
  int32_t tcond_dim = 0;
  Engine tgt, drf;                  // target denoiser; independent draft model (optional)
  bool has_drafter = false;
  int32_t picard_calls = 0;         // > 0: created for the Picard drafter
  std::vector<float> a_det, c_det;
  Layout lay{};
  char* ws = nullptr;
  size_t ws_bytes = 0;
  cudaStream_t stream = nullptr;
  uint64_t seed = 0;
  int64_t chain_off = 0;
  int32_t mode = SDS_FROZEN_PREV;
  State state = kCreated;
  int ub = 0;                       // host upper bound on active chains
  int last_cuda = 0;
  int64_t launches = 0;
  int32_t* h_pin = nullptr;         // pinned host words for the window loop
  cudaEvent_t ev[2] = {nullptr, nullptr};
  double tau = 1.0;                 // temperature of the accept test
  const float* Q = nullptr;         // orthonormal rows of the subspace the ratio is decided in (caller's)
  int32_t qr = 0;
  bool whole_chain = true;          // sds_sample_all may use the whole-chain kernel
  bool tensor_split = true;         // float mixtures of tensor-core shape use the 3-way bf16 split
  bool gemm_pair = true;            // tensor-core GEMMs with N % 256 == 0 run on CTA pairs
  bool early_exit = true;           // verify stops reading a window after the block with the first rejection
  bool fuse_advance = true;         // sds_sample_all lets the verify kernel do the advance step where it can
  bool regen = true;                // sds_sample_all lets the verify kernel draw the drafted states again instead of reading them
  bool regen_always = false;        // ... in every window (default: only while windows end after a few positions)
  bool fusing = false;              // set around the verify call of the sds_sample_all loop
  bool raw_rows = true;             // sds_sample_all lets the mixing GEMM store accumulators, verify applies C acc + E x
  bool onehot = true;               // the mixing GEMM skips blocks of rows that are all one-hot; a copy kernel fills them
  bool raw_now = false;             // set around the verify and advance calls of the sds_sample_all loop
  bool hot_now = false;             // likewise: rows of skipped (all one-hot) blocks are read from the means table, not stored
  bool regen_now = false;           // likewise: verify regenerates the drafted states
  bool skipx_now = false;           // likewise: the draft kernel stores only the bf16 copy of its rows
  int staged = 0;                   // SDS_OPT_STAGED_WINDOWS: 0 off, 1..L fixed stage length, SDS_STAGED_ADAPTIVE
  bool staged_now = false;          // set for the whole of a staged sds_sample_all
  int cap_now = 0, cap_next = 0;    // stage length of the window being enqueued, and of the one after it
  // optional per-kernel timing: event pairs recorded around each launch, summed on read
  bool prof_on = false;
  std::vector<cudaEvent_t> prof_ev[SDS_PROF_KINDS];
  size_t prof_used[SDS_PROF_KINDS] = {};
  double prof_ms[SDS_PROF_KINDS] = {};
  int64_t prof_n[SDS_PROF_KINDS] = {};
};

namespace {

// float mixture whose two contractions tile for the tensor cores (and is too large for the
// one-warp-per-row kernel): eligible for the split-precision path
bool gmm_split_shape(const sds_denoiser& den, int32_t d) {
  return den.kind == SDS_DEN_GMM && den.means_dtype == SDS_F32 && den.ncomp > 32 && den.ncomp % 128 == 0 &&
         den.ncomp <= 1024 && d % 128 == 0;
}

bool wants_bf16_rows(const sds_denoiser& den) {
  return den.kind == SDS_DEN_MLP || (den.kind == SDS_DEN_GMM && den.means_dtype == SDS_BF16);
}

void den_layout(Carve& cv, const sds_denoiser* den, size_t K, int tcond_dim, size_t rows, int32_t d, DenLayout* l) {
  l->tcond = cv.take(K * (size_t)(tcond_dim > 0 ? tcond_dim : 1) * 8);
  l->musq = (den->kind == SDS_DEN_GMM) ? cv.take((size_t)den->ncomp * 8) : kNone;
  l->H0 = l->H1 = l->logits = l->R = l->Mt = l->Xs = l->Ms = l->flags = l->amax = l->hot = kNone;
  if (gmm_split_shape(*den, d)) {
    l->Xs = cv.take(2 * rows * (size_t)d * 2);
    l->Ms = cv.take(3 * (size_t)den->ncomp * d * 2);
    l->Mt = cv.take(3 * (size_t)d * den->ncomp * 2);
    l->R = cv.take(3 * rows * (size_t)den->ncomp * 2);
    l->logits = cv.take(rows * (size_t)den->ncomp * 4);
    l->flags = cv.take(((rows + 255) / 256 * 2) * 4);
    l->amax = cv.take(rows * 4);
    l->hot = cv.take(((rows + 255) / 256 + 1) * 4);     // [0]: some block holds a row that is not one-hot; then one word per block
  }
  if (den->kind == SDS_DEN_MLP) {
    size_t width = 0;
    for (int i = 1; i < den->nlayer; ++i) width = std::max(width, (size_t)den->dims[i]);
    l->H0 = cv.take(rows * width * 2);
    l->H1 = cv.take(rows * width * 2);
  }
  if (den->kind == SDS_DEN_GMM && den->means_dtype == SDS_BF16) {
    l->logits = cv.take(rows * (size_t)den->ncomp * 4);
    l->R = cv.take(rows * (size_t)den->ncomp * 2);
    l->Mt = cv.take((size_t)d * den->ncomp * 2);
    l->amax = cv.take(rows * 4);
    l->hot = cv.take(((rows + 255) / 256 + 1) * 4);     // [0]: some block holds a row that is not one-hot; then one word per block
  }
}

void make_layout(const sds_schedule* sch, const sds_denoiser* den, const sds_denoiser* drafter, bool picard, int64_t B,
                 int32_t d, int32_t L, Layout* out, DenLayout* tl, DenLayout* dl) {
  Carve cv;
  Layout l{};
  const size_t K = (size_t)sch->K, rows = (size_t)B * L, Bd = (size_t)B * d;
  l.a = cv.take(K * 4);
  l.c = cv.take(K * 4);
  l.sigma = cv.take(K * 4);
  l.Y = cv.take(Bd * 4);
  l.Dc = cv.take(Bd * 4);
  l.T = cv.take(Bd * 4);
  l.X = cv.take(rows * d * 4);
  l.Dq = cv.take(rows * d * 4);
  l.Xb = wants_bf16_rows(*den) ? cv.take(rows * d * 2) : kNone;
  l.n = cv.take((size_t)B * 4);
  l.act = cv.take((size_t)B * 4);
  l.rowoff = cv.take((size_t)(B + 1) * 4);
  l.rowk = cv.take(rows * 4);
  l.ctl = cv.take(kCtlWords * 4);
  l.S1 = cv.take(rows * 8);
  l.S2 = cv.take(rows * 8);
  l.ell = cv.take(rows * 4);
  l.logU = cv.take(rows * 4);
  l.accmask = cv.take((size_t)B * 4);
  l.jstar = cv.take((size_t)B * 4);
  l.nfe_calls = cv.take((size_t)B * 4);
  l.nfe_rows = cv.take((size_t)B * 4);
  l.rem = cv.take((size_t)B * 4);
  den_layout(cv, den, K, sch->tcond_dim, rows, d, tl);
  tl->xb = l.Xb;
  l.Gx = l.Gb = l.Pb = l.Dp = l.Gk = kNone;
  if (drafter) {
    l.Gk = cv.take((size_t)B * 4);
    l.Gx = cv.take(Bd * 4);
    l.Gb = cv.take(Bd * 2);
    l.Pb = cv.take(Bd * 4);
    l.Dp = cv.take(rows * d * 4);
    den_layout(cv, drafter, K, 4, (size_t)B, d, dl);
    dl->xb = l.Gb;
  }
  l.ce = (den->kind == SDS_DEN_GMM) ? cv.take(K * 8) : kNone;
  l.adet = l.cdet = kNone;
  if (picard) {
    l.adet = cv.take(K * 4);
    l.cdet = cv.take(K * 4);
    l.Dp = cv.take(rows * d * 4);
  }
  l.total = cv.off;
  *out = l;
}

int validate_den(const sds_denoiser* den, const double* tcond, int tcond_dim, int32_t d);

int validate(const sds_schedule* sch, const sds_denoiser* den, int64_t B, int32_t d, int32_t L) {
  if (!sch || !den) return SDS_EINVAL;
  if (B <= 0 || d <= 0 || L < 1 || L > kMaxL || sch->K <= 0) return SDS_EINVAL;
  if (B * (int64_t)L > ((int64_t)1 << 30) || B > ((int64_t)1 << 30)) return SDS_EINVAL;
  if (!sch->a || !sch->c || !sch->sigma) return SDS_EINVAL;
  for (int k = 0; k < sch->K; ++k) {
    if (!std::isfinite(sch->a[k]) || !std::isfinite(sch->c[k]) || !std::isfinite(sch->sigma[k])) return SDS_EINVAL;
    if (!(sch->sigma[k] > 0.f)) return SDS_EINVAL;
  }
  return validate_den(den, sch->tcond, sch->tcond_dim, d);
}

int validate_den(const sds_denoiser* den, const double* tcond, int tcond_dim, int32_t d) {
  switch (den->kind) {
    case SDS_DEN_GMM:
      if (den->ncomp <= 0 || !den->means_dev || !den->logw_dev) return SDS_EINVAL;
      if (!tcond || tcond_dim != 4) return SDS_EINVAL;
      if (den->means_dtype == SDS_BF16) {
        // tensor-core path: both contractions tile by 128
        if (den->ncomp % 128 != 0 || d % 128 != 0) return SDS_EUNSUPPORTED;
      } else if (den->means_dtype != SDS_F32) {
        return SDS_EUNSUPPORTED;
      } else if (!gmm_f32_shape_ok(den->ncomp, d)) {
        return SDS_EUNSUPPORTED;          // more components than the float kernels hold logits for
      }
      break;
    case SDS_DEN_CALLBACK:
      if (!den->fn) return SDS_EINVAL;
      break;
    case SDS_DEN_PHI4:
      if (den->grid_side < 2 || (int64_t)den->grid_side * den->grid_side != d) return SDS_EINVAL;
      if (!std::isfinite(den->coupling)) return SDS_EINVAL;
      break;
    case SDS_DEN_MLP:
      if (den->nlayer < 1 || den->nlayer > 16 || !den->dims || !den->W_dev || !den->bias_dev || !den->temb_dev)
        return SDS_EINVAL;
      if (den->dims[0] != d || den->dims[den->nlayer] != d) return SDS_EINVAL;
      for (int i = 0; i <= den->nlayer; ++i)
        if (den->dims[i] <= 0 || den->dims[i] % 128 != 0) return SDS_EUNSUPPORTED;
      for (int i = 0; i < den->nlayer; ++i) {
        if (!den->W_dev[i] || !den->bias_dev[i]) return SDS_EINVAL;
        if (i < den->nlayer - 1 && !den->temb_dev[i]) return SDS_EINVAL;
      }
      break;
    default:
      return SDS_EUNSUPPORTED;
  }
  return SDS_OK;
}

template <class T>
T* at(sds_ctx* c, size_t off) { return off == kNone ? nullptr : reinterpret_cast<T*>(c->ws + off); }

WinArgs win_args(sds_ctx* c) {
  WinArgs A{};
  A.B = (int)c->B; A.d = c->d; A.L = c->L; A.K = c->K;
  A.mode = c->mode;
  A.inv_tau = 1.0 / c->tau;
  A.early_exit = c->early_exit ? 1 : 0;
  A.fuse_advance = c->fusing ? 1 : 0;
  A.raw_ce = c->raw_now ? at<float2>(c, c->lay.ce) : nullptr;
  if (c->hot_now) {
    A.hot_amax = at<int>(c, c->tgt.lay.amax);
    A.hot_flags = at<int>(c, c->tgt.lay.hot) + 1;       // (word 0 says whether any block is mixed)
    A.hot_means = c->tgt.den.means_dev;
    A.hot_bf16 = c->tgt.den.means_dtype == SDS_BF16 ? 1 : 0;
  }
  A.regen = c->regen_now ? 1 : 0;
  A.skip_x = c->skipx_now ? 1 : 0;
  A.staged = c->staged_now ? 1 : 0;
  A.cap = c->cap_now;
  A.cap_next = c->cap_next;
  A.rem = at<int>(c, c->lay.rem);
  A.seed = c->seed; A.chain_off = (uint64_t)c->chain_off;
  A.a = at<float>(c, c->lay.a); A.c = at<float>(c, c->lay.c); A.sigma = at<float>(c, c->lay.sigma);
  A.Y = at<float>(c, c->lay.Y); A.Dc = at<float>(c, c->lay.Dc); A.T = at<float>(c, c->lay.T);
  A.X = at<float>(c, c->lay.X); A.Dq = at<float>(c, c->lay.Dq); A.Xb = at<uint16_t>(c, c->lay.Xb);
  A.n = at<int>(c, c->lay.n); A.act = at<int>(c, c->lay.act); A.rowoff = at<int>(c, c->lay.rowoff);
  A.rowk = at<int>(c, c->lay.rowk); A.ctl = at<int>(c, c->lay.ctl);
  A.S1 = at<double>(c, c->lay.S1); A.S2 = at<double>(c, c->lay.S2);
  A.ell = at<float>(c, c->lay.ell); A.logU = at<float>(c, c->lay.logU);
  A.accmask = at<uint32_t>(c, c->lay.accmask); A.jstar = at<int>(c, c->lay.jstar);
  A.nfe_calls = at<int>(c, c->lay.nfe_calls); A.nfe_rows = at<int>(c, c->lay.nfe_rows);
  A.Gx = at<float>(c, c->lay.Gx); A.Gb = at<uint16_t>(c, c->lay.Gb); A.Gk = at<int>(c, c->lay.Gk);
  A.Pb = at<float>(c, c->lay.Pb); A.Dp = at<float>(c, c->lay.Dp);
  if (c->tensor_split && gmm_split_shape(c->tgt.den, c->d)) {   // draft and init write the row planes themselves
    A.Xs = at<uint16_t>(c, c->tgt.lay.Xs);
    A.xs_plane = (size_t)c->tgt.cap_rows * c->d;
  }
  A.Q = c->Q; A.qr = c->qr;
  A.mean_rows = c->mode == SDS_PICARD ? 1 : 0;
  A.picard_calls = c->picard_calls;
  A.a_det = at<float>(c, c->lay.adet); A.c_det = at<float>(c, c->lay.cdet);
  return A;
}

GmmArgs gmm_args(sds_ctx* c, Engine& e) {
  GmmArgs G{};
  G.d = c->d; G.ncomp = e.den.ncomp; G.K = c->K;
  G.tcond = at<double>(c, e.lay.tcond);
  G.means = static_cast<const float*>(e.den.means_dev);
  G.logw = e.den.logw_dev;
  G.musq = at<double>(c, e.lay.musq);
  return G;
}

int cuda_fail(sds_ctx* c, cudaError_t e) {
  c->last_cuda = (int)e;
  return SDS_ECUDA;
}
#define SDS_CU(ctx, expr)                                   \
  do {                                                      \
    cudaError_t e_ = (expr);                                \
    if (e_ != cudaSuccess) return cuda_fail((ctx), e_);     \
  } while (0)

// event pair around one launch of the given kind (only when profiling is on)
cudaError_t prof_mark(sds_ctx* c, int kind) {
  if (!c->prof_on) return cudaSuccess;
  std::vector<cudaEvent_t>& v = c->prof_ev[kind];
  if (c->prof_used[kind] == v.size()) {
    cudaEvent_t e;
    const cudaError_t rc = cudaEventCreate(&e);
    if (rc != cudaSuccess) return rc;
    v.push_back(e);
  }
  return cudaEventRecord(v[c->prof_used[kind]++], c->stream);
}

// fold finished event pairs into the sums (the stream must be idle)
void prof_collect(sds_ctx* c) {
  for (int k = 0; k < SDS_PROF_KINDS; ++k) {
    for (size_t i = 0; i + 1 < c->prof_used[k]; i += 2) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, c->prof_ev[k][i], c->prof_ev[k][i + 1]) == cudaSuccess) {
        c->prof_ms[k] += ms;
        c->prof_n[k] += 1;
      } else {
        cudaGetLastError();
      }
    }
    c->prof_used[k] = 0;
  }
}

#define SDS_LAUNCH(ctx, kind, expr)            \
  do {                                         \
    SDS_CU(ctx, prof_mark(ctx, kind));         \
    SDS_CU(ctx, expr);                         \
    SDS_CU(ctx, prof_mark(ctx, kind));         \
    (ctx)->launches++;                         \
  } while (0)

int ensure_musq(sds_ctx* c, Engine& e) {
  if (e.musq_ready) return SDS_OK;
  SDS_LAUNCH(c, SDS_PROF_AUX, launch_musq(static_cast<const float*>(e.den.means_dev), e.den.ncomp, c->d,
                                          at<double>(c, e.lay.musq), c->stream));
  e.musq_ready = true;
  return SDS_OK;
}

// bf16 copy of the rows for the tensor-core denoisers (the draft kernel writes it on the hot path)
int ensure_bf16_rows(sds_ctx* c, Engine& e, const float* X, const uint16_t** Xb, int64_t rows_ub) {
  if (*Xb) return SDS_OK;
  uint16_t* dst = at<uint16_t>(c, e.lay.xb);
  SDS_LAUNCH(c, &e == &c->drf ? SDS_PROF_DRAFT_MODEL : SDS_PROF_SOFTMAX, launch_f32_to_bf16(X, (size_t)rows_ub * c->d, dst, c->stream));
  *Xb = dst;
  return SDS_OK;
}

TcGemmArgs tc_args(sds_ctx* c, Engine& e, const int* rowk, const int* nrows_dev, int64_t rows_ub) {
  TcGemmArgs g{};
  g.nrows_dev = nrows_dev;
  g.rows_host = (int)rows_ub;
  g.rows_cap = (int)e.cap_rows;
  g.rowk = rowk;
  g.err = at<int>(c, c->lay.ctl) + kCtlTcError;
  g.pair = c->gemm_pair ? 1 : 0;
  return g;
}

// run the target denoiser on dense rows X (and their bf16 copy Xb, NULL = make one); the row count
// lives on the device (nrows_dev, may be NULL) with a host upper bound for the grids
int run_denoiser(sds_ctx* c, Engine& e, const float* X, const uint16_t* Xb, const int* rowk, const int* nrows_dev,
                 int64_t rows_ub, float* out, bool planes_ready = false, bool raw = false, bool indexed = false) {
  if (rows_ub <= 0) return SDS_OK;
  // timing kinds: the independent draft model's kernels are kept apart from the target's
  const bool is_drafter = &e == &c->drf;
  const int kd = is_drafter ? SDS_PROF_DRAFT_MODEL : SDS_PROF_DENOISE;
  const int ks = is_drafter ? SDS_PROF_DRAFT_MODEL : SDS_PROF_SOFTMAX;
  const int km = is_drafter ? SDS_PROF_DRAFT_MODEL : SDS_PROF_MIX;
  switch (e.den.kind) {
    case SDS_DEN_GMM: {
      if (e.den.means_dtype == SDS_F32 && c->tensor_split && gmm_split_shape(e.den, c->d)) {
        // Float mixture on the tensor cores: means and responsibilities are split into three bf16
        // planes each (x = h + m + l carries the 24-bit significand) and the mixing contraction
        // accumulates the six products of total order <= 2, smallest first, in one TMEM accumulator.
        // The logits only have to find the components within 30 of the row maximum (the softmax
        // kernel recomputes those in double; the rest weigh less than e^-29), so the rows are split in
        // two planes and three products (orders <= 1, a 16-bit significand) are enough.
        const float* means = static_cast<const float*>(e.den.means_dev);
        const size_t nc = (size_t)e.den.ncomp, dd = (size_t)c->d, cap = (size_t)e.cap_rows;
        uint16_t* Ms = at<uint16_t>(c, e.lay.Ms);
        uint16_t* Mt = at<uint16_t>(c, e.lay.Mt);
        uint16_t* Xs = at<uint16_t>(c, e.lay.Xs);
        uint16_t* Rs = at<uint16_t>(c, e.lay.R);
        float* logits = at<float>(c, e.lay.logits);
        const bool fresh = !e.musq_ready;
        int rc = ensure_musq(c, e);
        if (rc != SDS_OK) return rc;
        if (fresh) {
          SDS_LAUNCH(c, SDS_PROF_AUX, launch_split3(means, nc * dd, nc * dd, 3, Ms, c->stream));
          for (int i = 0; i < 3; ++i)
            SDS_LAUNCH(c, SDS_PROF_AUX, launch_transpose_bf16(Ms + i * nc * dd, (int)nc, (int)dd, Mt + i * nc * dd, c->stream));
        }
        if (!planes_ready)   // the draft and init kernels write the two row planes as they write the rows
          SDS_LAUNCH(c, ks, launch_split3(X, (size_t)rows_ub * dd, cap * dd, 2, Xs, c->stream));
        static const uint8_t kA[6] = {2, 1, 0, 1, 0, 0}, kB[6] = {0, 1, 2, 0, 1, 0};
        static const uint8_t kLa[3] = {1, 0, 0}, kLb[3] = {0, 1, 0};
        TcGemmArgs g = tc_args(c, e, rowk, nrows_dev, rows_ub);
        g.N = (int)nc; g.K = (int)dd; g.out = logits; g.ldo = (int)nc;
        g.tcond = at<double>(c, e.lay.tcond); g.musq = at<double>(c, e.lay.musq); g.logw = e.den.logw_dev;
        g.nseg = 3; g.nplanes = 2; g.a_plane = cap * dd; g.b_plane = nc * dd;
        for (int i = 0; i < 3; ++i) { g.a_idx[i] = kLa[i]; g.b_idx[i] = kLb[i]; }
        SDS_LAUNCH(c, kd, launch_gemm_tc(kEpiGmmLogits, g, Xs, Ms, c->stream));
        // rows whose responsibilities need only their first bf16 plane (one-hot rows above all) let
        // the mixing contraction drop the three products with the other planes, tile by tile
        int* flags = at<int>(c, e.lay.flags);
        SDS_CU(c, cudaMemsetAsync(flags, 0, (((size_t)rows_ub + 255) / 256 * 2) * 4, c->stream));
        // blocks of 256 rows whose rows are all one-hot skip the mixing contraction: their result is a copy of means
        int* amax = c->onehot ? at<int>(c, e.lay.amax) : nullptr;
        int* any_mixed = c->onehot ? at<int>(c, e.lay.hot) : nullptr;
        int* hot = any_mixed ? any_mixed + 1 : nullptr;
        if (hot) SDS_CU(c, cudaMemsetAsync(any_mixed, 0, (((size_t)rows_ub + 255) / 256 + 1) * 4, c->stream));
        SDS_LAUNCH(c, ks,
                   launch_softmax_split3(logits, nrows_dev, (int)rows_ub, (int)nc, (int)dd, X, means,
                                         at<double>(c, e.lay.musq), e.den.logw_dev, at<double>(c, e.lay.tcond), rowk,
                                         cap * nc, Rs, flags, amax, hot, any_mixed, c->stream));
        TcGemmArgs m = tc_args(c, e, rowk, nrows_dev, rows_ub);
        m.N = (int)dd; m.K = (int)nc; m.out = out; m.ldo = (int)dd;
        m.tcond = at<double>(c, e.lay.tcond); m.xrows = raw ? nullptr : X;
        m.nseg = 6; m.nplanes = 3; m.a_plane = cap * nc; m.b_plane = nc * dd;
        for (int i = 0; i < 6; ++i) { m.a_idx[i] = kA[i]; m.b_idx[i] = kB[i]; }
        static const uint8_t kSa[3] = {0, 0, 0}, kSb[3] = {2, 1, 0};   // the products with the first plane, same order
        m.tile_flags = flags; m.nseg_short = 3;
        m.tile_counts = at<int>(c, c->lay.ctl) + kCtlTilesFull;
        for (int i = 0; i < 3; ++i) { m.a_short[i] = kSa[i]; m.b_short[i] = kSb[i]; }
        m.hot_flags = hot; m.mixed_blocks = any_mixed;
        SDS_LAUNCH(c, km, launch_gemm_tc(kEpiGmmMix, m, Rs, Mt, c->stream));
        if (hot && !indexed)    // (indexed: the readers of the rows take the skipped blocks' rows from the means themselves)
          SDS_LAUNCH(c, ks, launch_mix_onehot(means, false, amax, hot, nrows_dev, (int)rows_ub, (int)dd,
                                              at<double>(c, e.lay.tcond), rowk, raw ? nullptr : X, out, c->stream));
        return SDS_OK;
      }
      if (e.den.means_dtype == SDS_F32) {
        const int rc = ensure_musq(c, e);
        if (rc != SDS_OK) return rc;
        SDS_LAUNCH(c, kd, launch_gmm_f32(gmm_args(c, e), X, rowk, nrows_dev, (int)rows_ub, out, c->stream));
        return SDS_OK;
      }
      // large mixture on tensor cores: logits = X M^T, softmax, mix = R M, affine epilogue
      const uint16_t* means = static_cast<const uint16_t*>(e.den.means_dev);
      uint16_t* Mt = at<uint16_t>(c, e.lay.Mt);
      uint16_t* R = at<uint16_t>(c, e.lay.R);
      float* logits = at<float>(c, e.lay.logits);
      if (!e.musq_ready) {
        SDS_LAUNCH(c, SDS_PROF_AUX, launch_musq_bf16(means, e.den.ncomp, c->d, at<double>(c, e.lay.musq), c->stream));
        SDS_LAUNCH(c, SDS_PROF_AUX, launch_transpose_bf16(means, e.den.ncomp, c->d, Mt, c->stream));
        e.musq_ready = true;
      }
      int rc = ensure_bf16_rows(c, e, X, &Xb, rows_ub);
      if (rc != SDS_OK) return rc;
      TcGemmArgs g = tc_args(c, e, rowk, nrows_dev, rows_ub);
      g.N = e.den.ncomp; g.K = c->d; g.out = logits; g.ldo = e.den.ncomp;
      g.tcond = at<double>(c, e.lay.tcond); g.musq = at<double>(c, e.lay.musq); g.logw = e.den.logw_dev;
      SDS_LAUNCH(c, kd, launch_gemm_tc(kEpiGmmLogits, g, Xb, means, c->stream));
      int* amax = c->onehot ? at<int>(c, e.lay.amax) : nullptr;
      int* any_mixed = c->onehot ? at<int>(c, e.lay.hot) : nullptr;
      int* hot = any_mixed ? any_mixed + 1 : nullptr;
      if (hot) SDS_CU(c, cudaMemsetAsync(any_mixed, 0, (((size_t)rows_ub + 255) / 256 + 1) * 4, c->stream));
      SDS_LAUNCH(c, ks, launch_softmax_bf16(logits, nrows_dev, (int)rows_ub, e.den.ncomp, R, amax, hot, any_mixed, c->stream));
      TcGemmArgs m = tc_args(c, e, rowk, nrows_dev, rows_ub);
      m.N = c->d; m.K = e.den.ncomp; m.out = out; m.ldo = c->d;
      m.tcond = at<double>(c, e.lay.tcond); m.xrows = raw ? nullptr : X;
      m.hot_flags = hot; m.mixed_blocks = any_mixed;
      m.tile_counts = is_drafter ? nullptr : at<int>(c, c->lay.ctl) + kCtlTilesFull;
      SDS_LAUNCH(c, km, launch_gemm_tc(kEpiGmmMix, m, R, Mt, c->stream));
      if (hot && !indexed)   // the skipped blocks: every row is a copy of one mean (with the same affine map as the epilogue's)
        SDS_LAUNCH(c, ks, launch_mix_onehot(means, true, amax, hot, nrows_dev, (int)rows_ub, c->d,
                                            at<double>(c, e.lay.tcond), rowk, raw ? nullptr : X, out, c->stream));
      return SDS_OK;
    }
    case SDS_DEN_MLP: {
      int rc = ensure_bf16_rows(c, e, X, &Xb, rows_ub);
      if (rc != SDS_OK) return rc;
      const void* in = Xb;
      const int nl = (int)e.mlp_W.size();
      for (int l = 0; l < nl; ++l) {
        TcGemmArgs g = tc_args(c, e, rowk, nrows_dev, rows_ub);
        g.N = e.mlp_dims[l + 1]; g.K = e.mlp_dims[l];
        g.bias = e.mlp_bias[l];
        if (l < nl - 1) {
          uint16_t* h = at<uint16_t>(c, (l & 1) ? e.lay.H1 : e.lay.H0);
          g.out = h; g.ldo = g.N; g.temb = static_cast<const uint16_t*>(e.mlp_temb[l]);
          SDS_LAUNCH(c, kd, launch_gemm_tc(kEpiMlpHidden, g, in, e.mlp_W[l], c->stream));
          in = h;
        } else {
          g.out = out; g.ldo = g.N;
          SDS_LAUNCH(c, kd, launch_gemm_tc(kEpiBiasF32, g, in, e.mlp_W[l], c->stream));
        }
      }
      return SDS_OK;
    }
    case SDS_DEN_PHI4:
      SDS_LAUNCH(c, kd, launch_phi4_grad(X, nrows_dev, (int)rows_ub, e.den.grid_side, e.den.coupling,
                                                        e.den.periodic, out, c->stream));
      return SDS_OK;
    case SDS_DEN_CALLBACK: {
      int32_t rows = (int32_t)rows_ub;         // the callback needs the row count on the host
      if (nrows_dev) {
        SDS_CU(c, cudaMemcpyAsync(c->h_pin + 4, nrows_dev, 4, cudaMemcpyDeviceToHost, c->stream));
        SDS_CU(c, cudaStreamSynchronize(c->stream));
        rows = c->h_pin[4];
      }
      if (rows <= 0) return SDS_OK;
      const int rc = e.den.fn(e.den.user, X, rowk, rows, c->d, out, (void*)c->stream);
      return rc == 0 ? SDS_OK : SDS_ECALLBACK;
    }
    default:
      return SDS_EUNSUPPORTED;
  }
}

int sync_active(sds_ctx* c, int64_t* n_active) {
  WinArgs A = win_args(c);
  SDS_CU(c, cudaMemcpyAsync(c->h_pin, A.ctl, kCtlWords * 4, cudaMemcpyDeviceToHost, c->stream));
  SDS_CU(c, cudaStreamSynchronize(c->stream));
  c->ub = c->h_pin[kCtlNActive];
  if (n_active) *n_active = c->ub;
  if (c->h_pin[kCtlTcError] != 0) return SDS_ETIMEOUT;
  return (c->h_pin[kCtlError] & kErrNonFinite) ? SDS_ENONFINITE : SDS_OK;
}

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

namespace {

void engine_init(Engine& e, const sds_denoiser* den, const double* tcond, int tcond_dim, int K, int64_t cap_rows) {
  e.den = *den;
  e.cap_rows = cap_rows;
  if (tcond && tcond_dim > 0) e.tcond.assign(tcond, tcond + (size_t)K * tcond_dim);
  if (den->kind == SDS_DEN_MLP) {
    e.mlp_dims.assign(den->dims, den->dims + den->nlayer + 1);
    e.mlp_W.assign(den->W_dev, den->W_dev + den->nlayer);
    e.mlp_bias.assign(den->bias_dev, den->bias_dev + den->nlayer);
    e.mlp_temb.assign(den->temb_dev, den->temb_dev + den->nlayer);
    e.den.dims = e.mlp_dims.data();
  }
}

struct PicardSpec {
  int32_t calls;
  const float* a_det;
  const float* c_det;
};

int create_impl(const sds_schedule* sch, const sds_denoiser* den, const sds_denoiser* drafter,
                const double* drafter_tcond, const PicardSpec* pic, int64_t B, int32_t d, int32_t L, sds_ctx** out,
                size_t* bytes_only) {
  int rc = validate(sch, den, B, d, L);
  if (rc != SDS_OK) return rc;
  if (pic && !bytes_only) {
    if (pic->calls < 1 || pic->calls > 64 || !pic->a_det || !pic->c_det) return SDS_EINVAL;
    for (int k = 0; k < sch->K; ++k)
      if (!std::isfinite(pic->a_det[k]) || !std::isfinite(pic->c_det[k])) return SDS_EINVAL;
  }
  if (drafter) {
    if (drafter->kind == SDS_DEN_CALLBACK) return SDS_EUNSUPPORTED;
    rc = validate_den(drafter, drafter_tcond, 4, d);
    if (rc != SDS_OK) return rc;
  }
  if (bytes_only) {
    Layout l;
    DenLayout tl, dl;
    make_layout(sch, den, drafter, pic != nullptr, B, d, L, &l, &tl, &dl);
    *bytes_only = l.total;
    return SDS_OK;
  }
  sds_ctx* c = new (std::nothrow) sds_ctx();
  if (!c) return SDS_ENOMEM;
  c->B = B; c->d = d; c->L = L; c->K = sch->K;
  c->a.assign(sch->a, sch->a + sch->K);
  c->c.assign(sch->c, sch->c + sch->K);
  c->sigma.assign(sch->sigma, sch->sigma + sch->K);
  c->tcond_dim = sch->tcond_dim > 0 ? sch->tcond_dim : 0;
  engine_init(c->tgt, den, sch->tcond, c->tcond_dim, sch->K, B * L);
  c->has_drafter = drafter != nullptr;
  if (drafter) engine_init(c->drf, drafter, drafter_tcond, 4, sch->K, B);
  if (pic) {
    c->picard_calls = pic->calls;
    c->a_det.assign(pic->a_det, pic->a_det + sch->K);
    c->c_det.assign(pic->c_det, pic->c_det + sch->K);
  }
  make_layout(sch, den, drafter, pic != nullptr, B, d, L, &c->lay, &c->tgt.lay, &c->drf.lay);
  if (cudaHostAlloc((void**)&c->h_pin, 64 * sizeof(int32_t), cudaHostAllocDefault) != cudaSuccess) {
    c->last_cuda = (int)cudaGetLastError();
    delete c;
    return SDS_ECUDA;
  }
  for (int i = 0; i < 2; ++i) {
    if (cudaEventCreateWithFlags(&c->ev[i], cudaEventDisableTiming) != cudaSuccess) {
      cudaGetLastError();
      if (i == 1) cudaEventDestroy(c->ev[0]);
      cudaFreeHost(c->h_pin);
      delete c;
      return SDS_ECUDA;
    }
  }
  *out = c;
  return SDS_OK;
}

}  // namespace

int sds_workspace_bytes(const sds_schedule* sch, const sds_denoiser* den, int64_t B, int32_t d, int32_t L,
                        size_t* bytes) {
  if (!bytes) return SDS_EINVAL;
  return create_impl(sch, den, nullptr, nullptr, nullptr, B, d, L, nullptr, bytes);
}

int sds_create(const sds_schedule* sch, const sds_denoiser* den, int64_t B, int32_t d, int32_t L, sds_ctx** out) {
  if (!out) return SDS_EINVAL;
  *out = nullptr;
  return create_impl(sch, den, nullptr, nullptr, nullptr, B, d, L, out, nullptr);
}

int sds_workspace_bytes_picard(const sds_schedule* sch, const sds_denoiser* den, int64_t B, int32_t d, int32_t L,
                               size_t* bytes) {
  if (!bytes) return SDS_EINVAL;
  const PicardSpec pic{1, nullptr, nullptr};
  return create_impl(sch, den, nullptr, nullptr, &pic, B, d, L, nullptr, bytes);
}

int sds_create_picard(const sds_schedule* sch, const sds_denoiser* den, int32_t calls, const float* a_det,
                      const float* c_det, int64_t B, int32_t d, int32_t L, sds_ctx** out) {
  if (!out) return SDS_EINVAL;
  *out = nullptr;
  const PicardSpec pic{calls, a_det, c_det};
  return create_impl(sch, den, nullptr, nullptr, &pic, B, d, L, out, nullptr);
}

int sds_workspace_bytes_with_drafter(const sds_schedule* sch, const sds_denoiser* den, const sds_denoiser* drafter,
                                     const double* drafter_tcond, int64_t B, int32_t d, int32_t L, size_t* bytes) {
  if (!bytes || !drafter) return SDS_EINVAL;
  return create_impl(sch, den, drafter, drafter_tcond, nullptr, B, d, L, nullptr, bytes);
}

int sds_create_with_drafter(const sds_schedule* sch, const sds_denoiser* den, const sds_denoiser* drafter,
                            const double* drafter_tcond, int64_t B, int32_t d, int32_t L, sds_ctx** out) {
  if (!out || !drafter) return SDS_EINVAL;
  *out = nullptr;
  return create_impl(sch, den, drafter, drafter_tcond, nullptr, B, d, L, out, nullptr);
}

int sds_bind(sds_ctx* c, void* workspace_dev, size_t bytes, void* cuda_stream, uint64_t seed, int32_t drafter_mode,
             int64_t chain_id_offset) {
  if (!c || !workspace_dev) return SDS_EINVAL;
  if (drafter_mode != SDS_FROZEN_PREV && drafter_mode != SDS_FROZEN_EXACT && drafter_mode != SDS_INDEPENDENT &&
      drafter_mode != SDS_PICARD)
    return SDS_EUNSUPPORTED;
  if ((drafter_mode == SDS_INDEPENDENT) != c->has_drafter) return SDS_EINVAL;   // the draft model and the mode go together
  if ((drafter_mode == SDS_PICARD) != (c->picard_calls > 0)) return SDS_EINVAL; // so do the Picard context and its mode
  if (chain_id_offset < 0) return SDS_EINVAL;
  if (bytes < c->lay.total || (reinterpret_cast<uintptr_t>(workspace_dev) % kAlign) != 0) return SDS_ENOMEM;
  c->ws = static_cast<char*>(workspace_dev);
  c->ws_bytes = bytes;
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  c->seed = seed;
  c->mode = drafter_mode;
  c->chain_off = chain_id_offset;
  c->tgt.musq_ready = c->drf.musq_ready = false;
  const size_t kb = (size_t)c->K * 4;
  SDS_CU(c, cudaMemcpyAsync(c->ws + c->lay.a, c->a.data(), kb, cudaMemcpyHostToDevice, c->stream));
  SDS_CU(c, cudaMemcpyAsync(c->ws + c->lay.c, c->c.data(), kb, cudaMemcpyHostToDevice, c->stream));
  SDS_CU(c, cudaMemcpyAsync(c->ws + c->lay.sigma, c->sigma.data(), kb, cudaMemcpyHostToDevice, c->stream));
  if (c->lay.ce != kNone && c->tgt.tcond.size() == (size_t)c->K * 4) {
    std::vector<float> ce((size_t)c->K * 2);
    for (int k = 0; k < c->K; ++k) {
      ce[2 * k] = (float)c->tgt.tcond[4 * (size_t)k + 2];
      ce[2 * k + 1] = (float)c->tgt.tcond[4 * (size_t)k + 3];
    }
    SDS_CU(c, cudaMemcpyAsync(c->ws + c->lay.ce, ce.data(), ce.size() * 4, cudaMemcpyHostToDevice, c->stream));
    SDS_CU(c, cudaStreamSynchronize(c->stream));      // the staging vector goes away
  }
  if (c->picard_calls > 0) {
    SDS_CU(c, cudaMemcpyAsync(c->ws + c->lay.adet, c->a_det.data(), kb, cudaMemcpyHostToDevice, c->stream));
    SDS_CU(c, cudaMemcpyAsync(c->ws + c->lay.cdet, c->c_det.data(), kb, cudaMemcpyHostToDevice, c->stream));
  }
  for (Engine* e : {&c->tgt, &c->drf})
    if (!e->tcond.empty())
      SDS_CU(c, cudaMemcpyAsync(c->ws + e->lay.tcond, e->tcond.data(), e->tcond.size() * 8, cudaMemcpyHostToDevice,
                                c->stream));
  SDS_CU(c, cudaMemsetAsync(c->ws + c->lay.ctl, 0, kCtlWords * 4, c->stream));
  SDS_CU(c, cudaStreamSynchronize(c->stream));
  c->state = kBound;
  return SDS_OK;
}

int sds_reset(sds_ctx* c) {
  if (!c) return SDS_EINVAL;
  if (c->state < kBound) return SDS_ESTATE;
  WinArgs A = win_args(c);
  SDS_LAUNCH(c, SDS_PROF_INIT, launch_init(A, c->stream));
  if (c->mode == SDS_FROZEN_PREV || c->mode == SDS_PICARD) {
    const int rc = run_denoiser(c, c->tgt, A.X, A.Xb, A.rowk, A.ctl + kCtlNRows, c->B, A.Dq, A.Xs != nullptr);
    if (rc != SDS_OK) return rc;
    SDS_LAUNCH(c, SDS_PROF_AUX, launch_after_init(A, c->stream));
  }
  SDS_LAUNCH(c, SDS_PROF_AUX, launch_compact(A, c->stream));
  c->ub = (int)c->B;
  c->state = kReady;
  return SDS_OK;
}

int sds_draft(sds_ctx* c) {
  if (!c) return SDS_EINVAL;
  if (c->state != kReady) return SDS_ESTATE;
  WinArgs A = win_args(c);
  if (c->mode == SDS_FROZEN_EXACT) {
    // frozen output = target output at (Y_n, t_n): one row per active chain
    SDS_LAUNCH(c, SDS_PROF_DRAFT, launch_gather_state(A, c->ub, c->stream));
    const int rc = run_denoiser(c, c->tgt, A.X, A.Xb, A.rowk, A.ctl + kCtlNActive, c->ub, A.Dq);
    if (rc != SDS_OK) return rc;
    SDS_LAUNCH(c, SDS_PROF_DRAFT, launch_scatter_carried(A, c->ub, c->stream));
  }
  if (c->mode == SDS_PICARD) {
    // the rows hold the deterministic sampler's points while the target refines them in parallel
    const int64_t rows_ub = (int64_t)c->ub * c->L;
    SDS_LAUNCH(c, SDS_PROF_DRAFT, launch_picard_start(A, c->ub, c->stream));
    for (int m = 1; m < c->picard_calls; ++m) {
      const int rc = run_denoiser(c, c->tgt, A.X, A.Xb, A.rowk, A.ctl + kCtlNRows, rows_ub, A.Dq);
      if (rc != SDS_OK) return rc;
      SDS_LAUNCH(c, SDS_PROF_DRAFT, launch_picard_step(A, c->ub, c->stream));
    }
    const int rc = run_denoiser(c, c->tgt, A.X, A.Xb, A.rowk, A.ctl + kCtlNRows, rows_ub, A.Dq);
    if (rc != SDS_OK) return rc;
    SDS_LAUNCH(c, SDS_PROF_DRAFT, launch_picard_draft(A, c->ub, c->stream));
  } else if (c->mode == SDS_INDEPENDENT) {
    // sequential draft: position j needs the draft model at W_{j-1}
    for (int j = 1; j <= c->L; ++j) {
      SDS_LAUNCH(c, SDS_PROF_DRAFT, launch_gather_pos(A, j, c->ub, c->stream));
      const int rc = run_denoiser(c, c->drf, A.Gx, A.Gb, A.Gk, A.ctl + kCtlNActive, c->ub, A.Pb);
      if (rc != SDS_OK) return rc;
      SDS_LAUNCH(c, SDS_PROF_DRAFT, launch_draft_pos(A, j, c->ub, c->stream));
    }
  } else {
    SDS_LAUNCH(c, SDS_PROF_DRAFT, launch_draft(A, c->ub, c->stream));
  }
  c->state = kDrafted;
  return SDS_OK;
}

int sds_verify_window(sds_ctx* c) {
  if (!c) return SDS_EINVAL;
  if (c->state != kDrafted) return SDS_ESTATE;
  WinArgs A = win_args(c);
  // rows drafted by k_draft (the two frozen-output modes) come with their bf16 planes
  const bool planes_ready = A.Xs != nullptr && (c->mode == SDS_FROZEN_PREV || c->mode == SDS_FROZEN_EXACT);
  // (the host's bound on the rows: a staged window has at most cap rows per chain)
  const int64_t rows_ub = (int64_t)c->ub * (c->staged_now ? std::min(c->cap_now, c->L) : c->L);
  const int rc = run_denoiser(c, c->tgt, A.X, A.Xb, A.rowk, A.ctl + kCtlNRows, rows_ub, A.Dq, planes_ready,
                              c->raw_now, c->hot_now);
  if (rc != SDS_OK) return rc;
  SDS_LAUNCH(c, SDS_PROF_VERIFY, launch_verify(A, c->ub, c->stream));
  c->state = kVerified;
  return SDS_OK;
}

int sds_advance(sds_ctx* c, int64_t* n_active) {
  if (!c) return SDS_EINVAL;
  if (c->state != kVerified) return SDS_ESTATE;
  SDS_LAUNCH(c, SDS_PROF_ADVANCE, launch_advance(win_args(c), c->ub, c->stream));
  c->state = kReady;
  if (n_active) return sync_active(c, n_active);
  return SDS_OK;
}

int sds_sample_all(sds_ctx* c, float* out_dev, int32_t* nfe_calls_dev, int32_t* nfe_rows_dev) {
  if (!c || !out_dev) return SDS_EINVAL;
  if (c->state < kBound) return SDS_ESTATE;
  WinArgs A = win_args(c);
  int rc = SDS_OK;
  if (c->whole_chain && !c->Q && (c->mode == SDS_FROZEN_PREV || c->mode == SDS_FROZEN_EXACT) &&
      c->tgt.den.kind == SDS_DEN_GMM && fused_small_supported(c->d, c->tgt.den.ncomp, c->L)) {
    if ((rc = ensure_musq(c, c->tgt)) != SDS_OK) return rc;
    SDS_CU(c, cudaMemsetAsync(A.ctl, 0, kCtlWords * 4, c->stream));   // no chain active afterwards, error bits clear
    SDS_LAUNCH(c, SDS_PROF_FUSED, launch_fused_small(A, gmm_args(c, c->tgt), nullptr, c->stream));
    c->ub = 0;
    c->state = kReady;
  } else if (c->whole_chain && !c->Q && c->mode == SDS_INDEPENDENT && c->tgt.den.kind == SDS_DEN_GMM &&
             c->tgt.den.means_dtype == SDS_F32 && c->drf.den.kind == SDS_DEN_GMM && c->drf.den.means_dtype == SDS_F32 &&
             fused_small_supported_with_drafter(c->d, c->tgt.den.ncomp, c->drf.den.ncomp, c->L)) {
    // small target and small independent draft model: both mixtures live in shared memory
    if ((rc = ensure_musq(c, c->tgt)) != SDS_OK) return rc;
    if ((rc = ensure_musq(c, c->drf)) != SDS_OK) return rc;
    SDS_CU(c, cudaMemsetAsync(A.ctl, 0, kCtlWords * 4, c->stream));
    const GmmArgs gd = gmm_args(c, c->drf);
    SDS_LAUNCH(c, SDS_PROF_FUSED, launch_fused_small(A, gmm_args(c, c->tgt), &gd, c->stream));
    c->ub = 0;
    c->state = kReady;
  } else if (c->whole_chain && !c->Q && c->mode == SDS_FROZEN_EXACT && c->tgt.den.kind == SDS_DEN_PHI4 &&
             fused_phi4_ok(c->d, c->L)) {
    SDS_CU(c, cudaMemsetAsync(A.ctl, 0, kCtlWords * 4, c->stream));
    SDS_LAUNCH(c, SDS_PROF_FUSED, launch_fused_phi4(A, c->tgt.den.grid_side, c->tgt.den.coupling, c->tgt.den.periodic, c->stream));
    c->ub = 0;
    c->state = kReady;
  } else {
    // Staged windows: a launch drafts and verifies at most `cap` positions of every chain's window; a chain whose
    // stage accepted everything goes on with the rest of its window in the next launch, its carried output still
    // frozen, so the samples are those of whole windows, bit for bit, while the rows that follow a rejection are
    // never drafted nor given to the target. The stage length follows the share of chain-stages that passed.
    struct StageGuard {
      sds_ctx* c;
      ~StageGuard() { c->staged_now = false; }
    } stage_guard{c};
    const bool adaptive = c->staged == SDS_STAGED_ADAPTIVE;
    c->staged_now = c->staged != 0 && c->mode == SDS_FROZEN_PREV && !c->Q;
    c->cap_now = c->cap_next = (c->staged_now && !adaptive) ? std::min(c->staged, c->L) : c->L;
    int cap_hist[2] = {c->cap_now, c->cap_now};
    int cap_policy = c->cap_next;                        // the stage length the next enqueued scan will be given
    int64_t passed_seen = 0;
    rc = sds_reset(c);
    if (rc != SDS_OK) return rc;
    // Windows are enqueued one ahead of the host's knowledge of the active count: after window w
    // is enqueued the host waits for window w-1's count. A window enqueued with no active chain
    // does nothing on the device.
    // positions per chain the last known window evaluated (with early exit: up to the first rejection): decides,
    // window by window, whether verify makes the drafted states again or reads them back
    double mean_positions = (double)c->L;
    int64_t pos_seen = 0;
    int na_before = (int)c->B;
    for (int w = 0;; ++w) {
      // mixtures on the tensor cores: the mixing GEMM stores its accumulators and the verify (and advance)
      // kernels, which hold the rows' inputs anyway, apply C acc + E x: the GEMM's epilogue reads nothing
      const bool tensor_mix = c->tgt.den.kind == SDS_DEN_GMM &&
                              (c->tgt.den.means_dtype == SDS_BF16 || (c->tensor_split && gmm_split_shape(c->tgt.den, c->d)));
      c->raw_now = c->raw_rows && tensor_mix && (c->mode == SDS_FROZEN_PREV || c->mode == SDS_FROZEN_EXACT) &&
                   verify_reads_raw_rows(A);
      // ... and where every row of a block of 256 is one-hot, the block's accumulators are rows of the means table:
      // nothing is stored for it, verify and advance read the means
      c->hot_now = c->raw_now && c->onehot;
      // Frozen drafter whose target reads nothing but the bf16 copy of its input rows (the MLP; the bf16 mixture
      // with raw rows): the draft kernel stores only that copy, and verify, which then has no float rows to
      // read, makes the drafted states again from what it holds and advances its chains (it alone knows the
      // accepted state). Drawing the noise again costs about as much as reading the rows would, so this pays
      // only through the draft kernel's smaller writes; where the float rows are needed anyway it stays off.
      const bool bf16_only = A.Xb != nullptr &&
                             (c->tgt.den.kind == SDS_DEN_MLP ||
                              (c->tgt.den.kind == SDS_DEN_GMM && c->tgt.den.means_dtype == SDS_BF16 && c->raw_now));
      // Windows in which most drafts pass are verified over many positions, and there reading the drafted rows
      // back is cheaper than drawing their noise a second time; windows that end after a position or two (the
      // usual case late in a diffusion chain) gain from the smaller draft stores. The two ways give the same
      // bits, so the choice follows the positions per chain the latest finished window needed.
      const bool few_positions = !c->early_exit || mean_positions <= 0.25 * c->L + 1.0;
      c->regen_now = c->regen && c->fuse_advance && bf16_only && verify_can_regen(A) && (c->regen_always || few_positions);
      c->skipx_now = c->regen_now;
      // where the register-resident verify kernel runs, it also advances its chains and compacts
      c->fusing = c->fuse_advance && (verify_can_advance(A) || c->regen_now);
      c->cap_now = c->cap_next;                          // what the last scan sized this window's rows for
      c->cap_next = cap_policy;                          // what this window's scan sizes the next window's rows for
      cap_hist[w & 1] = c->cap_now;
      if (w == 0) {                                      // which of these paths the run may take (read back with the control words)
        const bool may_regen = c->regen && c->fuse_advance && bf16_only && verify_can_regen(A);
        c->h_pin[48] = (may_regen ? 1 : 0) | (c->hot_now ? 4 : 0);
        SDS_CU(c, cudaMemcpyAsync(A.ctl + kCtlPathFlags, c->h_pin + 48, 4, cudaMemcpyHostToDevice, c->stream));
      }
      rc = sds_draft(c);
      if (rc != SDS_OK) { c->fusing = c->raw_now = c->hot_now = c->regen_now = c->skipx_now = false; return rc; }
      rc = sds_verify_window(c);
      const bool fused_adv = c->fusing;
      c->fusing = false;
      if (rc == SDS_OK) {
        if (fused_adv) c->state = kReady;
        else rc = sds_advance(c, nullptr);
      }
      c->raw_now = c->hot_now = c->regen_now = c->skipx_now = false;
      if (rc != SDS_OK) return rc;
      SDS_CU(c, cudaMemcpyAsync(c->h_pin + 16 + (w & 1) * kCtlWords, A.ctl, kCtlWords * 4, cudaMemcpyDeviceToHost,
                                c->stream));
      SDS_CU(c, cudaEventRecord(c->ev[w & 1], c->stream));
      if (w >= 1) {
        SDS_CU(c, cudaEventSynchronize(c->ev[(w - 1) & 1]));
        const int32_t* seen = c->h_pin + 16 + ((w - 1) & 1) * kCtlWords;
        const int na = seen[kCtlNActive];
        if (na == 0) break;
        const int64_t pos = (int64_t)(uint32_t)seen[kCtlPositions];
        if (na_before > 0) mean_positions = (double)(pos - pos_seen) / na_before;
        pos_seen = pos;
        if (c->staged_now && adaptive && na_before > 0) {
          // window w-1 ran with cap_hist[(w-1)&1]; the scan of window w is enqueued already, so the new length
          // reaches window w+2
          const double pass = (double)((int64_t)(uint32_t)seen[kCtlStagePassed] - passed_seen) / na_before;
          const int used = cap_hist[(w - 1) & 1];
          if (pass > 0.5) cap_policy = std::min(c->L, std::max(cap_policy, 2 * used));
          else if (pass < 0.125) cap_policy = std::max(1, std::min(cap_policy, used / 2));
        }
        passed_seen = (int64_t)(uint32_t)seen[kCtlStagePassed];
        na_before = na;
        c->ub = na;
      }
      if (w > c->K + 2) break;   // every window advances each active chain by at least one step
    }
  }
  const size_t Bd = (size_t)c->B * c->d;
  if (out_dev != A.Y) SDS_CU(c, cudaMemcpyAsync(out_dev, A.Y, Bd * 4, cudaMemcpyDeviceToDevice, c->stream));
  if (nfe_calls_dev)
    SDS_CU(c, cudaMemcpyAsync(nfe_calls_dev, A.nfe_calls, (size_t)c->B * 4, cudaMemcpyDeviceToDevice, c->stream));
  if (nfe_rows_dev)
    SDS_CU(c, cudaMemcpyAsync(nfe_rows_dev, A.nfe_rows, (size_t)c->B * 4, cudaMemcpyDeviceToDevice, c->stream));
  int64_t na = 0;
  return sync_active(c, &na);
}

int sds_sample_all_host(sds_ctx* c, const void* means_host, const float* logw_host, float* out_host,
                        int32_t* nfe_calls_host, int32_t* nfe_rows_host) {
  if (!c || !out_host) return SDS_EINVAL;
  if (c->state < kBound) return SDS_ESTATE;
  if ((means_host || logw_host) && c->tgt.den.kind != SDS_DEN_GMM) return SDS_EINVAL;
  if (means_host) {
    const size_t esz = c->tgt.den.means_dtype == SDS_BF16 ? 2 : 4;
    SDS_CU(c, cudaMemcpyAsync(const_cast<void*>(c->tgt.den.means_dev), means_host, (size_t)c->tgt.den.ncomp * c->d * esz,
                              cudaMemcpyHostToDevice, c->stream));
    c->tgt.musq_ready = false;
  }
  if (logw_host)
    SDS_CU(c, cudaMemcpyAsync(const_cast<float*>(c->tgt.den.logw_dev), logw_host, (size_t)c->tgt.den.ncomp * 4,
                              cudaMemcpyHostToDevice, c->stream));
  WinArgs A = win_args(c);
  const int rc = sds_sample_all(c, A.Y, nullptr, nullptr);
  if (rc != SDS_OK && rc != SDS_ENONFINITE) return rc;
  SDS_CU(c, cudaMemcpyAsync(out_host, A.Y, (size_t)c->B * c->d * 4, cudaMemcpyDeviceToHost, c->stream));
  if (nfe_calls_host)
    SDS_CU(c, cudaMemcpyAsync(nfe_calls_host, A.nfe_calls, (size_t)c->B * 4, cudaMemcpyDeviceToHost, c->stream));
  if (nfe_rows_host)
    SDS_CU(c, cudaMemcpyAsync(nfe_rows_host, A.nfe_rows, (size_t)c->B * 4, cudaMemcpyDeviceToHost, c->stream));
  SDS_CU(c, cudaStreamSynchronize(c->stream));
  return rc;
}

int sds_get(sds_ctx* c, int32_t what, void* dst, size_t bytes, int32_t dst_is_host) {
  if (!c || !dst) return SDS_EINVAL;
  if (c->state < kBound) return SDS_ESTATE;
  const size_t B = (size_t)c->B, rows = B * c->L, d = (size_t)c->d;
  size_t off = 0, len = 0;
  switch (what) {
    case SDS_GET_X: off = c->lay.X; len = rows * d * 4; break;
    case SDS_GET_TAIL: off = c->lay.T; len = B * d * 4; break;
    case SDS_GET_DQ: off = c->lay.Dq; len = rows * d * 4; break;
    case SDS_GET_DC: off = c->lay.Dc; len = B * d * 4; break;
    case SDS_GET_Y: off = c->lay.Y; len = B * d * 4; break;
    case SDS_GET_N: off = c->lay.n; len = B * 4; break;
    case SDS_GET_ACT: off = c->lay.act; len = B * 4; break;
    case SDS_GET_ROWOFF: off = c->lay.rowoff; len = (B + 1) * 4; break;
    case SDS_GET_S1: off = c->lay.S1; len = rows * 8; break;
    case SDS_GET_S2: off = c->lay.S2; len = rows * 8; break;
    case SDS_GET_ELL: off = c->lay.ell; len = rows * 4; break;
    case SDS_GET_LOGU: off = c->lay.logU; len = rows * 4; break;
    case SDS_GET_ACCMASK: off = c->lay.accmask; len = B * 4; break;
    case SDS_GET_JSTAR: off = c->lay.jstar; len = B * 4; break;
    case SDS_GET_NFE_CALLS: off = c->lay.nfe_calls; len = B * 4; break;
    case SDS_GET_NFE_ROWS: off = c->lay.nfe_rows; len = B * 4; break;
    case SDS_GET_CTL: off = c->lay.ctl; len = kCtlWords * 4; break;
    case SDS_GET_ROWK: off = c->lay.rowk; len = rows * 4; break;
    case SDS_GET_DP:
      if (c->lay.Dp == kNone) return SDS_EINVAL;
      off = c->lay.Dp; len = rows * d * 4; break;
    default: return SDS_EINVAL;
  }
  if (bytes > len) return SDS_EINVAL;
  SDS_CU(c, cudaMemcpyAsync(dst, c->ws + off, bytes, dst_is_host ? cudaMemcpyDeviceToHost : cudaMemcpyDeviceToDevice,
                            c->stream));
  if (dst_is_host) SDS_CU(c, cudaStreamSynchronize(c->stream));
  return SDS_OK;
}

int sds_set_state(sds_ctx* c, const float* Y_dev, const int32_t* n_dev, const float* Dc_dev) {
  if (!c) return SDS_EINVAL;
  if (c->state != kReady) return SDS_ESTATE;
  const size_t Bd = (size_t)c->B * c->d * 4;
  if (Y_dev) SDS_CU(c, cudaMemcpyAsync(c->ws + c->lay.Y, Y_dev, Bd, cudaMemcpyDeviceToDevice, c->stream));
  if (Dc_dev) SDS_CU(c, cudaMemcpyAsync(c->ws + c->lay.Dc, Dc_dev, Bd, cudaMemcpyDeviceToDevice, c->stream));
  if (n_dev)
    SDS_CU(c, cudaMemcpyAsync(c->ws + c->lay.n, n_dev, (size_t)c->B * 4, cudaMemcpyDeviceToDevice, c->stream));
  SDS_CU(c, cudaMemsetAsync(c->ws + c->lay.rem, 0, (size_t)c->B * 4, c->stream));   // no window is under way
  SDS_LAUNCH(c, SDS_PROF_AUX, launch_compact(win_args(c), c->stream));
  c->ub = (int)c->B;
  return SDS_OK;
}

int sds_denoise(sds_ctx* c, const float* x_dev, const int32_t* k_dev, int64_t rows, float* out_dev) {
  if (!c || !x_dev || !k_dev || !out_dev) return SDS_EINVAL;
  if (c->state < kBound) return SDS_ESTATE;
  if (rows < 0 || rows > c->B * c->L) return SDS_EINVAL;
  return run_denoiser(c, c->tgt, x_dev, nullptr, k_dev, nullptr, rows, out_dev);
}

int sds_rng_normals(uint64_t seed, int32_t stream_id, int64_t b0, int64_t nb, int32_t k, int32_t d, float* out_dev,
                    void* cuda_stream) {
  if (!out_dev || nb < 0 || d <= 0 || k < 0 || b0 < 0) return SDS_EINVAL;
  if (nb == 0) return SDS_OK;
  return launch_rng_normals(seed, stream_id, (uint64_t)b0, nb, k, d, out_dev, (cudaStream_t)cuda_stream) == cudaSuccess
             ? SDS_OK
             : SDS_ECUDA;
}

int sds_rng_uniforms(uint64_t seed, int64_t b0, int64_t nb, int32_t k, float* u_dev, void* cuda_stream) {
  if (!u_dev || nb < 0 || k < 0 || b0 < 0) return SDS_EINVAL;
  if (nb == 0) return SDS_OK;
  return launch_rng_uniforms(seed, (uint64_t)b0, nb, k, u_dev, (cudaStream_t)cuda_stream) == cudaSuccess ? SDS_OK
                                                                                                           : SDS_ECUDA;
}

int sds_selftest_bounded_wait(int32_t polls, int32_t* status_dev, void* cuda_stream) {
  if (!status_dev || polls <= 0 || polls > (1 << 24)) return SDS_EINVAL;
  return launch_wait_selftest((uint32_t)polls, status_dev, (cudaStream_t)cuda_stream) == cudaSuccess ? SDS_OK
                                                                                                       : SDS_ECUDA;
}

int64_t sds_launch_count(const sds_ctx* c) { return c ? c->launches : 0; }

int sds_set_option(sds_ctx* c, int32_t option, int64_t value) {
  if (!c) return SDS_EINVAL;
  switch (option) {
    case SDS_OPT_WHOLE_CHAIN_KERNEL: c->whole_chain = value != 0; return SDS_OK;
    case SDS_OPT_TENSOR_SPLIT: c->tensor_split = value != 0; return SDS_OK;
    case SDS_OPT_GEMM_PAIR: c->gemm_pair = value != 0; return SDS_OK;
    case SDS_OPT_VERIFY_EARLY_EXIT: c->early_exit = value != 0; return SDS_OK;
    case SDS_OPT_FUSE_ADVANCE: c->fuse_advance = value != 0; return SDS_OK;
    case SDS_OPT_RAW_ROWS: c->raw_rows = value != 0; return SDS_OK;
    case SDS_OPT_REGEN_DRAFTS: c->regen = value != 0; c->regen_always = value == 2; return SDS_OK;
    case SDS_OPT_ONEHOT_ROWS: c->onehot = value != 0; return SDS_OK;
    case SDS_OPT_STAGED_WINDOWS:
      if (value < 0 || (value > 32 && value != SDS_STAGED_ADAPTIVE)) return SDS_EINVAL;
      c->staged = (int)value;
      return SDS_OK;
    default: return SDS_EINVAL;
  }
}

int sds_set_temperature(sds_ctx* c, double tau) {
  if (!c || !(tau > 0.0) || !std::isfinite(tau)) return SDS_EINVAL;
  c->tau = tau;
  return SDS_OK;
}

int sds_set_projection(sds_ctx* c, const float* Q_dev, int32_t r) {
  if (!c || r < 0 || (Q_dev && r == 0) || (!Q_dev && r != 0)) return SDS_EINVAL;
  if (Q_dev && (r > c->d || c->d > 16384)) return SDS_EUNSUPPORTED;
  c->Q = Q_dev;
  c->qr = r;
  return SDS_OK;
}

int sds_profile(sds_ctx* c, int32_t enable) {
  if (!c) return SDS_EINVAL;
  if (c->state >= kBound) SDS_CU(c, cudaStreamSynchronize(c->stream));
  prof_collect(c);
  c->prof_on = enable != 0;
  return SDS_OK;
}

int sds_profile_read(sds_ctx* c, double* ms, int64_t* launches, int32_t reset) {
  if (!c || !ms || !launches) return SDS_EINVAL;
  if (c->state >= kBound) SDS_CU(c, cudaStreamSynchronize(c->stream));
  prof_collect(c);
  for (int k = 0; k < SDS_PROF_KINDS; ++k) {
    ms[k] = c->prof_ms[k];
    launches[k] = c->prof_n[k];
    if (reset) { c->prof_ms[k] = 0.0; c->prof_n[k] = 0; }
  }
  return SDS_OK;
}

const char* sds_strerror(int code) {
  switch (code) {
    case SDS_OK: return "ok";
    case SDS_EINVAL: return "invalid argument";
    case SDS_ESTATE: return "call out of order";
    case SDS_ENOMEM: return "workspace too small or misaligned";
    case SDS_EUNSUPPORTED: return "unsupported configuration";
    case SDS_ECUDA: return "CUDA error";
    case SDS_ETIMEOUT: return "device-side wait timed out";
    case SDS_ENONFINITE: return "non-finite log ratio: chain frozen";
    case SDS_ECALLBACK: return "denoiser callback failed";
    default: return "unknown error";
  }
}

int sds_last_cuda_error(const sds_ctx* c) { return c ? c->last_cuda : 0; }

void sds_destroy(sds_ctx* c) {
  if (!c) return;
  for (int i = 0; i < 2; ++i)
    if (c->ev[i]) cudaEventDestroy(c->ev[i]);
  for (int k = 0; k < SDS_PROF_KINDS; ++k)
    for (cudaEvent_t e : c->prof_ev[k]) cudaEventDestroy(e);
  if (c->h_pin) cudaFreeHost(c->h_pin);
  delete c;
}

#pragma GCC visibility pop
}  // extern "C"
