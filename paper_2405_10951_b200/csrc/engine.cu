// Step engine and C ABI of the BSR fine-tuning step (see include/bsr.h for the contract).
//
// The engine carves one caller-owned workspace into: parameters in the storage dtype, fp32 master /
// gradient / AdamW moments of the trainable parameters (flat arrays), the activations the trainable
// blocks keep for their backward pass, and scratch shared by all blocks.  Frozen blocks write nothing
// that outlives them (paper Fig. 2: gradient propagation stops at the earliest trainable block).
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <string>
#include <vector>

#include "../../include/bsr.h"
#include "common.cuh"
#include "kernels.h"

using namespace bsr;

namespace {

thread_local char g_error[256] = "no error";

struct Schedule {
  int ta[BSR_MAX_DEPTH], tf[BSR_MAX_DEPTH], k[BSR_MAX_DEPTH];
};

struct Tensor {
  std::string name;
  size_t numel = 0;
  bool matrix = false;      // stored in the storage dtype; vectors (biases, LayerNorm, cls, pos) stay float
  bool trainable = false;
  bool decay = false;
  size_t w_off = 0;         // byte offset of the stored copy (for trainable float tensors: inside master)
  size_t flat = 0;          // element offset in the flat trainable arrays
};

struct BlockBufs {          // byte offsets into the workspace; filled for frozen (scratch) and trainable (arena) blocks
  size_t x_in, y1, qkv, o, xp_full, xp, y2, z, hh, x_out;
  size_t mean1, rstd1, lse, mean2, rstd2, p, s, kept, dropped;
  size_t o_cls, xin_cls;    // classification rows of o and of the block input (last block only)
  // MoE blocks: routing tables and expert-ordered buffers
  size_t m_eidx, m_ew, m_pos, m_row_token, m_row_w, m_seg, m_tile, m_cnt, m_off, m_xg, m_zg, m_hg, m_og;
};

// Carves the workspace.  Every slice is followed by a guard of GUARD_BYTES holding a fixed pattern; bsr_sync_status
// checks the guards, so a kernel that writes past the end of its slice is reported instead of silently corrupting the
// neighbour (the stand-in for a memory checker).
constexpr size_t GUARD_BYTES = 256;
constexpr uint32_t GUARD_WORD = 0xC5A3C5A3u;
struct Bump {
  size_t off = 0;
  std::vector<size_t>* guards = nullptr;
  size_t take(size_t bytes) {
    size_t o = off;
    off += (bytes + 255) & ~(size_t)255;
    if (guards != nullptr) guards->push_back(off);
    off += GUARD_BYTES;
    return o;
  }
};

int set_err(char* buf, int code, const char* fmt, ...) __attribute__((format(printf, 3, 4)));
int set_err(char* buf, int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, 256, fmt, ap);
  va_end(ap);
  return code;
}

int compute_schedule(const bsr_config* cfg, Schedule* s, char* err) {
  const bsr_dims& d = cfg->dims;
  if (d.patch_size <= 0 || d.image_size <= 0 || d.image_size % d.patch_size != 0)
    return set_err(err, BSR_ERR_INVALID_ARG, "image_size must be a positive multiple of patch_size");
  if (d.depth < 1 || d.depth > BSR_MAX_DEPTH) return set_err(err, BSR_ERR_INVALID_ARG, "depth must be in [1, %d]", BSR_MAX_DEPTH);
  if (cfg->n_drop < 0 || cfg->n_drop > BSR_MAX_DROPS) return set_err(err, BSR_ERR_INVALID_ARG, "n_drop must be in [0, %d]", BSR_MAX_DROPS);
  int g = d.image_size / d.patch_size;
  int t = g * g + 1;
  int di = 0;
  for (int i = 0; i < cfg->n_drop; ++i) {
    if (cfg->drop_block[i] < 0 || cfg->drop_block[i] >= d.depth || (i > 0 && cfg->drop_block[i] <= cfg->drop_block[i - 1]))
      return set_err(err, BSR_ERR_INVALID_ARG, "drop_block must be strictly ascending block indices");
    if (cfg->keep_den[i] <= 0 || cfg->keep_num[i] <= 0 || cfg->keep_num[i] > cfg->keep_den[i])
      return set_err(err, BSR_ERR_INVALID_ARG, "keep rate must satisfy 0 < keep_num <= keep_den");
  }
  for (int l = 0; l < d.depth; ++l) {
    s->ta[l] = t;
    s->k[l] = -1;
    if (di < cfg->n_drop && cfg->drop_block[di] == l) {
      long m = t - 1;
      long k = ((long)cfg->keep_num[di] * m + cfg->keep_den[di] - 1) / cfg->keep_den[di];   // ceil(keep * M)
      if (k < 1) k = 1;
      if (k > m) k = m;
      s->k[l] = (int)k;
      if (k < m) t = 1 + (int)k + (cfg->fuse_mode != BSR_FUSE_NONE ? 1 : 0);
      ++di;
    }
    s->tf[l] = t;
  }
  return BSR_OK;
}

int validate(const bsr_config* cfg, char* err) {
  if (cfg == nullptr) return set_err(err, BSR_ERR_INVALID_ARG, "config is null");
  const bsr_dims& d = cfg->dims;
  if (d.dtype != BSR_DTYPE_FP32 && d.dtype != BSR_DTYPE_BF16) return set_err(err, BSR_ERR_INVALID_ARG, "dtype must be fp32 (0) or bf16 (1)");
  if (d.in_chans < 1 || d.dim < 8 || d.heads < 1 || d.mlp_hidden < 8) return set_err(err, BSR_ERR_INVALID_ARG, "bad model dimension");
  if (d.dim % d.heads != 0) return set_err(err, BSR_ERR_INVALID_ARG, "dim must be a multiple of heads");
  if (d.dim % 8 != 0 || d.mlp_hidden % 8 != 0 || d.dim > 1024) return set_err(err, BSR_ERR_INVALID_ARG, "dim and mlp_hidden must be multiples of 8, dim <= 1024");
  int hd = d.dim / d.heads;
  if (hd > 64 || hd % 8 != 0) return set_err(err, BSR_ERR_INVALID_ARG, "head dimension must be a multiple of 8, at most 64");
  if (d.num_tasks < 1 || d.num_tasks > BSR_MAX_TASKS) return set_err(err, BSR_ERR_INVALID_ARG, "num_tasks must be in [1, %d]", BSR_MAX_TASKS);
  for (int t = 0; t < d.num_tasks; ++t)
    if (d.num_classes[t] < 1) return set_err(err, BSR_ERR_INVALID_ARG, "num_classes must be positive");
  if (cfg->max_batch < 1) return set_err(err, BSR_ERR_INVALID_ARG, "max_batch must be positive");
  if (cfg->fuse_mode != BSR_FUSE_NONE && cfg->fuse_mode != BSR_FUSE_WEIGHTED_SUM && cfg->fuse_mode != BSR_FUSE_WEIGHTED_MEAN)
    return set_err(err, BSR_ERR_INVALID_ARG, "unknown fuse_mode");
  if (cfg->optimizer != BSR_OPT_ADAMW && cfg->optimizer != BSR_OPT_SGD) return set_err(err, BSR_ERR_INVALID_ARG, "unknown optimizer");
  if (cfg->optimizer == BSR_OPT_SGD && !(cfg->momentum >= 0.f && cfg->momentum < 1.f)) return set_err(err, BSR_ERR_INVALID_ARG, "momentum must lie in [0, 1)");
  if (!(d.ln_eps > 0.f)) return set_err(err, BSR_ERR_INVALID_ARG, "ln_eps must be positive");
  if (cfg->frozen_fp8 != 0 && cfg->frozen_fp8 != 1) return set_err(err, BSR_ERR_INVALID_ARG, "frozen_fp8 must be 0 or 1");
  if (cfg->frozen_fp8 && (d.dtype != BSR_DTYPE_BF16 || d.dim % 16 != 0))
    return set_err(err, BSR_ERR_UNSUPPORTED, "the 8-bit prefix needs a bf16 model whose dim is a multiple of 16");
  Schedule s;
  int rc = compute_schedule(cfg, &s, err);
  if (rc != BSR_OK) return rc;
  if (d.depth < 32 && (cfg->trainable_mask >> d.depth) != 0) return set_err(err, BSR_ERR_INVALID_ARG, "trainable_mask names a block beyond depth");
  if (d.moe_block_mask != 0) {
    if (d.depth < 32 && (d.moe_block_mask >> d.depth) != 0) return set_err(err, BSR_ERR_INVALID_ARG, "moe_block_mask names a block beyond depth");
    if (d.moe_experts < 1 || d.moe_experts > 32 || d.moe_top_k < 1 || d.moe_top_k > 4 || d.moe_top_k > d.moe_experts)
      return set_err(err, BSR_ERR_INVALID_ARG, "MoE needs 1 <= experts <= 32 and 1 <= top_k <= min(4, experts)");
    if (d.dtype != BSR_DTYPE_BF16) return set_err(err, BSR_ERR_UNSUPPORTED, "MoE layers run on the bf16 tensor-core kernels only");
    if (d.dim % 64 != 0 || d.mlp_hidden % 64 != 0) return set_err(err, BSR_ERR_UNSUPPORTED, "MoE layers need dim and mlp_hidden to be multiples of 64");
  }
  return BSR_OK;
}

}  // namespace

struct bsr_handle {
  bsr_config cfg;
  Schedule sched;
  char* base = nullptr;
  size_t bytes = 0;
  char err[256];
  int sm_count = 148;
  int use_tc = 1;
  int64_t step = 0;
  float lr = 0.f;
  int t0 = 0;                        // earliest trainable block (depth if none)
  std::vector<Tensor> tensors;
  std::map<std::string, int> index;
  size_t n_flat = 0;                 // elements in the flat trainable arrays
  size_t off_status = 0, off_loss = 0;
  size_t off_weights = 0, weights_bytes = 0;
  size_t off_frozen_vec = 0;
  size_t off_master = 0, off_grad = 0, off_m = 0, off_v = 0;
  size_t off_chunks = 0;
  int n_chunks = 0;
  std::vector<BlockBufs> bufs_train;  // per block (valid for l >= t0)
  BlockBufs bufs_frozen[2];           // ping-pong by block parity
  size_t off_x_last = 0;
  size_t arena_bytes = 0, scratch_bytes = 0;
  size_t block_saved_bytes[BSR_MAX_DEPTH] = {};
  // scratch
  size_t off_patches = 0, off_emb = 0;
  size_t off_xn = 0, off_meanf = 0, off_rstdf = 0, off_logits = 0, off_per_image = 0, off_dlogits = 0, off_dxn = 0;
  size_t off_dxa = 0, off_dxb = 0, off_dz = 0, off_dy = 0, off_dxg = 0, off_dxp = 0, off_do = 0, off_dqkv = 0;
  size_t off_dxa_c = 0, off_dxb_c = 0, off_dxg_c = 0, off_dxp_c = 0;
  size_t off_escore = 0, off_delta = 0, off_ln_partials = 0, off_cs_partials = 0;
  size_t off_kept_all = 0;
  size_t off_stage = 0;
  size_t off_split = 0, split_floats = 0;
  std::vector<size_t> moe_rec_eidx, moe_rec_ew;
  std::vector<size_t> score_rec;       // per drop location's block: head-mean scores [max_batch, M] of the last step
  size_t off_m_dog = 0, off_m_dzg = 0, off_m_dxg = 0, off_m_dw = 0, off_m_dsel = 0;
  GemmProfile prof;
  // Captured graphs of the training step.  The key is everything a captured launch has baked in: the caller's
  // pointers, the batch, the kernel mode and whether the step reads its inputs through the multi-step loop state.
  // Up to GRAPH_CACHE graphs are kept; the least recently used one is dropped.
  struct StepGraph { const void* images; const void* labels; const void* tasks; void* loss; void* kept; int batch; int mode; int loop;
                     cudaGraphExec_t exec; long launches; uint64_t last_use; };
  static constexpr size_t GRAPH_CACHE = 8;
  std::vector<StepGraph> graphs;
  uint64_t graph_clock = 0;
  uint64_t graph_captures = 0;        // how many times a step was captured (a pipeline that cycles through more buffers than the cache holds re-captures every step)
  int use_graph = 1;
  // multi-step loop and host-buffer step
  // E4M3 copies of the QKV and first-FFN weights of the dense blocks before t0 (frozen_fp8), with a scale per row
  std::vector<size_t> q_qkv, q_qkv_s, q_fc1, q_fc1_s;
  size_t off_yq = 0, off_yq_s = 0;        // LayerNorm output as E4M3 rows and their scales
  std::vector<size_t> guards;            // byte offsets of the guard words after every slice
  size_t off_guard_table = 0;
  size_t off_loop = 0, off_lab_stage = 0, off_task_stage = 0;
  size_t off_host_img[2] = {0, 0}, off_host_lab[2] = {0, 0}, off_host_task[2] = {0, 0}, off_host_loss[2] = {0, 0};
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_copied[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr};
  bool slot_used[2] = {false, false};
  int host_slot = 0;
  SideLane side;                        // second lane for the reductions only the optimiser reads
  int use_side = 1;
  long launches_at_enable = 0;

  template <typename T> T* at(size_t off) const { return reinterpret_cast<T*>(base + off); }
  void* w(const char* name) const {
    auto it = index.find(name);
    return it == index.end() ? nullptr : base + tensors[it->second].w_off;
  }
  void* wb(int l, const char* suffix) const { return w(("blocks." + std::to_string(l) + "." + suffix).c_str()); }
  float* gradp(const std::string& name) const {
    auto it = index.find(name);
    return at<float>(off_grad) + tensors[it->second].flat;
  }
  float* gb(int l, const char* suffix) const { return gradp("blocks." + std::to_string(l) + "." + suffix); }
};

namespace {

void build_tensors(bsr_handle* h) {
  const bsr_dims& d = h->cfg.dims;
  int D = d.dim, F = d.mlp_hidden;
  int g = d.image_size / d.patch_size;
  auto add = [&](const std::string& name, size_t numel, bool matrix, bool trainable) {
    Tensor t;
    t.name = name; t.numel = numel; t.matrix = matrix; t.trainable = trainable;
    t.decay = name.size() >= 6 && name.compare(name.size() - 6, 6, "weight") == 0 && name.find("norm") == std::string::npos;
    h->index[name] = (int)h->tensors.size();
    h->tensors.push_back(t);
  };
  add("patch_embed.weight", (size_t)D * d.in_chans * d.patch_size * d.patch_size, true, false);
  add("patch_embed.bias", D, false, false);
  add("cls_token", D, false, false);
  add("pos_embed", (size_t)(g * g + 1) * D, false, false);
  for (int l = 0; l < d.depth; ++l) {
    bool tr = (h->cfg.trainable_mask >> l) & 1u;
    std::string p = "blocks." + std::to_string(l) + ".";
    add(p + "norm1.weight", D, false, tr);
    add(p + "norm1.bias", D, false, tr);
    add(p + "attn.qkv.weight", (size_t)3 * D * D, true, tr);
    add(p + "attn.qkv.bias", 3 * D, false, tr);
    add(p + "attn.proj.weight", (size_t)D * D, true, tr);
    add(p + "attn.proj.bias", D, false, tr);
    add(p + "norm2.weight", D, false, tr);
    add(p + "norm2.bias", D, false, tr);
    if ((d.moe_block_mask >> l) & 1u) {
      size_t E = d.moe_experts;
      add(p + "moe.gate.weight", (size_t)d.num_tasks * E * D, true, tr);
      add(p + "moe.fc1.weight", E * F * D, true, tr);
      add(p + "moe.fc1.bias", E * F, false, tr);
      add(p + "moe.fc2.weight", E * D * F, true, tr);
      add(p + "moe.fc2.bias", E * D, false, tr);
    } else {
      add(p + "mlp.fc1.weight", (size_t)F * D, true, tr);
      add(p + "mlp.fc1.bias", F, false, tr);
      add(p + "mlp.fc2.weight", (size_t)D * F, true, tr);
      add(p + "mlp.fc2.bias", D, false, tr);
    }
  }
  add("norm.weight", D, false, true);
  add("norm.bias", D, false, true);
  for (int t = 0; t < d.num_tasks; ++t) {
    add("head." + std::to_string(t) + ".weight", (size_t)d.num_classes[t] * D, true, true);
    add("head." + std::to_string(t) + ".bias", d.num_classes[t], false, true);
  }
}

constexpr uint32_t ADAM_CHUNK = 4096;

// Lays the workspace out; identical for sizing (base == nullptr) and for creation.
size_t plan(bsr_handle* h) {
  const bsr_config& cfg = h->cfg;
  const bsr_dims& d = cfg.dims;
  const Schedule& s = h->sched;
  size_t es = dtype_size(d.dtype);
  int D = d.dim, F = d.mlp_hidden, H = d.heads, Bm = cfg.max_batch;
  int g = d.image_size / d.patch_size, N = g * g, T0 = N + 1;
  int cmax = 0;
  for (int t = 0; t < d.num_tasks; ++t) cmax = d.num_classes[t] > cmax ? d.num_classes[t] : cmax;
  Bump b;
  h->guards.clear();
  b.guards = &h->guards;
  h->off_status = b.take(256);
  h->off_loss = h->off_status + 64;
  // flat trainable arrays
  size_t flat = 0;
  for (auto& t : h->tensors)
    if (t.trainable) { t.flat = flat; flat += (t.numel + 63) & ~(size_t)63; }
  h->n_flat = flat;
  h->off_master = b.take(flat * 4);
  h->off_grad = b.take(flat * 4);
  h->off_m = b.take(flat * 4);
  h->off_v = b.take(flat * 4);
  // stored copies
  size_t w0 = b.off;
  for (auto& t : h->tensors) {
    bool alias_master = t.trainable && (!t.matrix || d.dtype == BSR_DTYPE_FP32);
    if (alias_master) t.w_off = h->off_master + t.flat * 4;
    else t.w_off = b.take(t.numel * (t.matrix ? es : 4));
  }
  h->off_weights = w0;
  h->weights_bytes = b.off - w0;
  // AdamW chunk table
  int nch = 0;
  for (auto& t : h->tensors)
    if (t.trainable) nch += (int)((t.numel + ADAM_CHUNK - 1) / ADAM_CHUNK);
  h->n_chunks = nch;
  h->off_chunks = b.take((size_t)nch * sizeof(AdamChunk));
  // 8-bit copies of the gradient-free prefix's LayerNorm-fed weights
  h->t0 = cfg.trainable_mask ? __builtin_ctz(cfg.trainable_mask) : d.depth;
  h->q_qkv.assign(d.depth, 0); h->q_qkv_s.assign(d.depth, 0); h->q_fc1.assign(d.depth, 0); h->q_fc1_s.assign(d.depth, 0);
  if (cfg.frozen_fp8)
    for (int l = 0; l < h->t0 && l < d.depth; ++l) {
      if ((d.moe_block_mask >> l) & 1u) continue;
      h->q_qkv[l] = b.take((size_t)3 * D * D); h->q_qkv_s[l] = b.take((size_t)3 * D * 4);
      h->q_fc1[l] = b.take((size_t)F * D); h->q_fc1_s[l] = b.take((size_t)F * 4);
    }
  h->weights_bytes = b.off - w0;
  // routing record of every MoE block (kept for inspection), then the activations kept by the trainable blocks
  int E = d.moe_experts, Kx = d.moe_top_k;
  std::vector<size_t> rec_eidx(d.depth, 0), rec_ew(d.depth, 0);
  for (int l = 0; l < d.depth; ++l)
    if ((d.moe_block_mask >> l) & 1u) {
      rec_eidx[l] = b.take((size_t)Bm * s.tf[l] * Kx * 4);
      rec_ew[l] = b.take((size_t)Bm * s.tf[l] * Kx * 4);
    }
  auto take_moe = [&](BlockBufs& bb, int l, size_t tokens_ffn) {
    size_t M = (size_t)Bm * tokens_ffn;
    size_t cap = (size_t)moe_rows_cap((int)M, E, Kx);
    bb.m_eidx = rec_eidx[l];
    bb.m_ew = rec_ew[l];
    bb.m_pos = b.take(M * Kx * 4);
    bb.m_row_token = b.take(cap * 4);
    bb.m_row_w = b.take(cap * 4);
    bb.m_seg = b.take((size_t)(E + 1) * 4);
    bb.m_tile = b.take((cap / 128) * 4);
    bb.m_cnt = b.take((size_t)moe_blocks((int)M) * E * 4);
    bb.m_off = b.take((size_t)moe_blocks((int)M) * E * 4);
    bb.m_xg = b.take(cap * D * es);
    bb.m_zg = b.take(cap * F * es);
    bb.m_hg = b.take(cap * F * es);
    bb.m_og = b.take(cap * D * 4);
  };
  h->moe_rec_eidx = rec_eidx;
  h->moe_rec_ew = rec_ew;
  // head-mean scores of every drop location (Eq. 6), kept for inspection whether the block is frozen or trains
  h->score_rec.assign(d.depth, 0);
  for (int l = 0; l < d.depth; ++l)
    if (s.k[l] >= 0) h->score_rec[l] = b.take((size_t)Bm * (s.ta[l] - 1) * 4);
  // activations kept by the trainable blocks
  size_t a0 = b.off;
  h->bufs_train.assign(d.depth, BlockBufs());
  h->t0 = cfg.trainable_mask ? __builtin_ctz(cfg.trainable_mask) : d.depth;
  size_t next_in = 0;
  for (int l = h->t0; l < d.depth; ++l) {
    BlockBufs& bb = h->bufs_train[l];
    size_t Ma = (size_t)Bm * s.ta[l], Mf = (size_t)Bm * s.tf[l];
    bool drop = s.k[l] >= 0 && s.tf[l] != s.ta[l];
    size_t block0 = b.off;
    bb.x_in = (l == h->t0) ? b.take(Ma * D * 4) : next_in;       // residual stream: float
    // A trainable block keeps the input of every linear layer (Eq. 4: its weight gradient needs it); a frozen block
    // inside the gradient path keeps only what passing the gradient on needs (Eq. 2; Section 3.2, Table 1): Q, K, V
    // with the log-sum-exp, the FFN pre-activation, and the LayerNorm inputs with their statistics.  Its LayerNorm
    // outputs and attention output live in the scratch the blocks before t0 use.  The GELU output is kept by no block:
    // the backward pass recomputes it from the pre-activation where the second FFN layer's weight gradient needs it.
    bool keeps_inputs = (cfg.trainable_mask >> l) & 1u;
    bb.mean1 = b.take(Ma * 4); bb.rstd1 = b.take(Ma * 4);
    bb.y1 = keeps_inputs ? b.take(Ma * D * es) : 0;
    bb.qkv = b.take(Ma * 3 * D * es);
    bb.lse = b.take((size_t)Bm * H * s.ta[l] * 4);
    bb.o = keeps_inputs ? b.take(Ma * D * es) : 0;
    bb.xp = b.take(Mf * D * 4);
    bb.xp_full = drop ? b.take(Ma * D * 4) : bb.xp;
    if (s.k[l] >= 0) {
      bb.p = b.take((size_t)Bm * H * (s.ta[l] - 1) * 4);
      bb.s = h->score_rec[l];
      bb.kept = b.take((size_t)Bm * (s.ta[l] - 1) * 4);
      bb.dropped = b.take((size_t)Bm * (s.ta[l] - 1) * 4);
    }
    bb.mean2 = b.take(Mf * 4); bb.rstd2 = b.take(Mf * 4);
    bb.y2 = keeps_inputs ? b.take(Mf * D * es) : 0;
    bool moe = (d.moe_block_mask >> l) & 1u;
    bb.z = moe ? 0 : b.take(Mf * F * es);
    bb.hh = 0;
    bb.x_out = b.take(Mf * D * 4);
    bb.o_cls = b.take((size_t)Bm * D * es);
    bb.xin_cls = b.take((size_t)Bm * D * 4);
    if (moe) take_moe(bb, l, s.tf[l]);
    next_in = bb.x_out;
    h->block_saved_bytes[l] = b.off - block0;
  }
  h->arena_bytes = b.off - a0;
  // scratch
  size_t s0 = b.off;
  size_t M0 = (size_t)Bm * T0;
  h->off_patches = b.take((size_t)Bm * N * d.in_chans * d.patch_size * d.patch_size * es);
  h->off_emb = b.take((size_t)Bm * N * D * es);
  size_t xa = b.take(M0 * D * 4), xb = b.take(M0 * D * 4);
  for (int i = 0; i < 2; ++i) {
    BlockBufs& bb = h->bufs_frozen[i];
    bb.x_in = i == 0 ? xa : xb;
    bb.x_out = i == 0 ? xb : xa;
  }
  {
    BlockBufs& bb = h->bufs_frozen[0];
    bb.mean1 = bb.rstd1 = bb.mean2 = bb.rstd2 = bb.lse = 0;
    bb.y1 = b.take(M0 * D * es);
    bb.qkv = b.take(M0 * 3 * D * es);
    bb.o = b.take(M0 * D * es);
    bb.xp_full = b.take(M0 * D * 4);
    bb.xp = b.take(M0 * D * 4);
    bb.y2 = bb.y1;
    bb.z = 0;
    bb.hh = b.take(M0 * F * es);
    bb.p = b.take((size_t)Bm * H * (T0 - 1) * 4);
    bb.s = b.take((size_t)Bm * (T0 - 1) * 4);
    bb.kept = b.take((size_t)Bm * (T0 - 1) * 4);
    bb.dropped = b.take((size_t)Bm * (T0 - 1) * 4);
    bb.o_cls = b.take((size_t)Bm * D * es);
    bb.xin_cls = b.take((size_t)Bm * D * 4);
    if (d.moe_block_mask != 0) take_moe(bb, 0, T0);          // frozen MoE blocks share one set sized for the longest sequence
    size_t in1 = h->bufs_frozen[1].x_in, out1 = h->bufs_frozen[1].x_out;
    h->bufs_frozen[1] = bb;
    h->bufs_frozen[1].x_in = in1;
    h->bufs_frozen[1].x_out = out1;
    // what the blocks from t0 on do not keep lives in the same scratch
    for (int l = h->t0; l < d.depth; ++l) {
      BlockBufs& tb = h->bufs_train[l];
      tb.hh = bb.hh;
      if (!((cfg.trainable_mask >> l) & 1u)) { tb.y1 = bb.y1; tb.o = bb.o; tb.y2 = bb.y2; }
    }
  }
  if (cfg.frozen_fp8) {
    h->off_yq = b.take(M0 * D);
    h->off_yq_s = b.take(M0 * 4);
  }
  h->off_xn = b.take((size_t)Bm * D * 4);
  h->off_meanf = b.take((size_t)Bm * 4);
  h->off_rstdf = b.take((size_t)Bm * 4);
  h->off_logits = b.take((size_t)Bm * cmax * 4);
  h->off_per_image = b.take((size_t)Bm * 4);
  h->off_dlogits = b.take((size_t)Bm * cmax * 4);
  h->off_dxn = b.take((size_t)Bm * D * 4);
  size_t kept_total = 0;
  for (int l = 0; l < d.depth; ++l)
    if (s.k[l] >= 0) kept_total += (size_t)Bm * s.k[l];
  h->off_kept_all = b.take((kept_total + 1) * 4);
  if (h->t0 < d.depth) {
    size_t Mt = (size_t)Bm * s.ta[h->t0];
    h->off_dxa = b.take(Mt * D * 4);            // gradient of the residual stream: float ...
    h->off_dxb = b.take(Mt * D * 4);
    h->off_dxg = b.take(Mt * D * 4);
    h->off_dxp = b.take(Mt * D * 4);
    if (d.dtype == BSR_DTYPE_BF16) {            // ... with a bf16 copy as GEMM operand
      h->off_dxa_c = b.take(Mt * D * es);
      h->off_dxb_c = b.take(Mt * D * es);
      h->off_dxg_c = b.take(Mt * D * es);
      h->off_dxp_c = b.take(Mt * D * es);
    }
    h->off_dz = b.take(Mt * F * es);
    h->off_dy = b.take(Mt * D * es);
    h->off_do = b.take(Mt * D * es);
    h->off_dqkv = b.take(Mt * 3 * D * es);
    h->off_escore = b.take((size_t)Bm * s.ta[h->t0] * 4);
    h->off_delta = b.take((size_t)Bm * H * s.ta[h->t0] * 4);
  }
  if (d.moe_block_mask != 0 && h->t0 < d.depth) {
    size_t cap = (size_t)moe_rows_cap(Bm * s.tf[h->t0], E, Kx);
    h->off_m_dog = b.take(cap * D * es);
    h->off_m_dzg = b.take(cap * F * es);
    h->off_m_dxg = b.take(cap * D * es);
    h->off_m_dw = b.take(cap * 4);
    h->off_m_dsel = b.take(cap * 4);
  }
  int maxn = 3 * D > F ? 3 * D : F;
  h->off_ln_partials = b.take((size_t)3 * 512 * D * 4);
  h->off_cs_partials = b.take((size_t)64 * maxn * 4);
  size_t biggest = 0;
  for (auto& t : h->tensors) biggest = t.numel > biggest ? t.numel : biggest;
  h->off_stage = b.take(biggest * 4);
  h->split_floats = (d.dtype == BSR_DTYPE_BF16) ? (size_t)160 * 128 * 256 : 0;   // one 128x256 fp32 tile per SM
  h->off_split = b.take(h->split_floats * 4);
  // multi-step loop state and staging; two staging slots for steps fed from host memory
  h->off_loop = b.take(256);
  h->off_lab_stage = b.take((size_t)Bm * 4);
  h->off_task_stage = b.take((size_t)Bm * 4);
  for (int i = 0; i < 2; ++i) {
    h->off_host_img[i] = b.take((size_t)Bm * d.in_chans * d.image_size * d.image_size * es);
    h->off_host_lab[i] = b.take((size_t)Bm * 4);
    h->off_host_task[i] = b.take((size_t)Bm * 4);
    h->off_host_loss[i] = b.take(256);
  }
  h->scratch_bytes = b.off - s0;
  // table of the guard offsets, read by the kernels that write and check the guards (it has no guard of its own)
  b.guards = nullptr;
  h->off_guard_table = b.take(h->guards.size() * sizeof(unsigned long long));
  return b.off;
}

Ctx make_ctx(const bsr_handle* h, void* stream) {
  Ctx c;
  c.stream = (cudaStream_t)stream;
  c.dtype = h->cfg.dims.dtype;
  c.status = h->at<int>(h->off_status);
  c.sm_count = h->sm_count;
  c.use_tc = h->use_tc;
  c.split_ws = h->split_floats ? h->at<float>(h->off_split) : nullptr;
  c.split_ws_floats = h->split_floats;
  c.prof = const_cast<GemmProfile*>(&h->prof);
  c.side = (h->use_side && h->side.stream != nullptr && !h->prof.on) ? const_cast<SideLane*>(&h->side) : nullptr;
  return c;
}

int check_cuda(bsr_handle* h, const char* what) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return set_err(h ? h->err : g_error, BSR_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
  return BSR_OK;
}

// In the last block only the classification token's output is ever used (the head reads row 0), so everything
// after the attention product -- projection, LayerNorm 2, FFN and their backward -- runs on the B classification
// rows alone.  The results are identical: the other rows' outputs feed nothing and their gradients are zero.
bool cls_tail(const bsr_handle* h, int l) { return l == h->cfg.dims.depth - 1 && h->sched.k[l] < 0; }

// One encoder block forward.  `save` keeps the statistics and pre-activations the backward pass needs.
bool is_moe(const bsr_handle* h, int l) { return (h->cfg.dims.moe_block_mask >> l) & 1u; }

MoeBufs moe_bufs(const bsr_handle* h, const BlockBufs& bb) {
  MoeBufs m;
  m.eidx = h->at<int>(bb.m_eidx); m.ew = h->at<float>(bb.m_ew); m.pos = h->at<int>(bb.m_pos);
  m.row_token = h->at<int>(bb.m_row_token); m.row_w = h->at<float>(bb.m_row_w);
  m.seg_start = h->at<int>(bb.m_seg); m.tile_expert = h->at<int>(bb.m_tile);
  m.blk_counts = h->at<int>(bb.m_cnt); m.blk_off = h->at<int>(bb.m_off);
  m.xg = h->base + bb.m_xg; m.zg = h->base + bb.m_zg; m.hg = h->base + bb.m_hg; m.og = h->at<float>(bb.m_og);
  return m;
}

int block_forward(bsr_handle* h, const Ctx& c, int l, int B, const BlockBufs& bb, bool save, int* kept_out, const int* task_ids) {
  const bsr_dims& d = h->cfg.dims;
  const Schedule& s = h->sched;
  int D = d.dim, F = d.mlp_hidden, H = d.heads, hd = D / H;
  int Ta = s.ta[l], Tf = s.tf[l], k = s.k[l];
  int Ma = B * Ta, Mf = B * Tf;
  bool is_drop = k >= 0;
  bool shrinks = is_drop && Tf != Ta;
  Ctx cf = c;                // the residual stream is float whatever the storage dtype
  cf.dtype = 0;
  // gradient-free prefix with 8-bit operands: the LayerNorm output leaves as E4M3 rows and meets the E4M3 weight copy
  const bool fp8 = !save && l < h->t0 && h->cfg.frozen_fp8 && h->q_qkv[l] != 0 && c.use_tc;
  GemmEpilogue e1;
  e1.bias = (const float*)h->wb(l, "attn.qkv.bias");
  if (fp8) {
    layernorm_fwd_e4m3(c, h->at<float>(bb.x_in), D, (const float*)h->wb(l, "norm1.weight"), (const float*)h->wb(l, "norm1.bias"),
                       h->base + h->off_yq, h->at<float>(h->off_yq_s), Ma, D, d.ln_eps);
    if (gemm_tc_e4m3(c, h->base + h->off_yq, h->at<float>(h->off_yq_s), h->base + h->q_qkv[l], h->at<float>(h->q_qkv_s[l]),
                     h->base + bb.qkv, Ma, 3 * D, D, e1) != 0)
      return set_err(h->err, BSR_ERR_CUDA, "8-bit GEMM set-up failed");
  } else {
    layernorm_fwd(c, h->at<float>(bb.x_in), D, (const float*)h->wb(l, "norm1.weight"), (const float*)h->wb(l, "norm1.bias"),
                  h->base + bb.y1, 0, save ? h->at<float>(bb.mean1) : nullptr, save ? h->at<float>(bb.rstd1) : nullptr, Ma, D, d.ln_eps);
    gemm(c, h->base + bb.y1, D, 1, h->wb(l, "attn.qkv.weight"), D, 1, h->base + bb.qkv, 0, Ma, 3 * D, D, e1);
  }
  size_t es = dtype_size(d.dtype);
  bool tail = cls_tail(h, l);
  // the last block needs the classification query only (its other outputs feed nothing)
  bool cls_attn = tail && attention_cls_fwd(c, h->base + bb.qkv, h->base + bb.o_cls, B, Ta, H, hd) == 0;
  if (!cls_attn) {
    int rc = attention_fwd(c, h->base + bb.qkv, h->base + bb.o, save ? h->at<float>(bb.lse) : nullptr,
                           is_drop ? h->at<float>(bb.p) : nullptr, B, Ta, H, hd);
    if (rc != 0) return set_err(h->err, BSR_ERR_UNSUPPORTED, "attention: %d tokens of head dimension %d do not fit this kernel", Ta, hd);
  }
  const void* proj_in = h->base + bb.o;
  const void* proj_res = h->base + bb.x_in;
  if (tail) {                  // from here on: B rows
    if (!cls_attn) copy_rows(c.stream, h->base + bb.o, (long)Ta * D * es, h->base + bb.o_cls, (long)D * es, B, (int)(D * es));
    copy_rows(c.stream, h->base + bb.x_in, (long)Ta * D * 4, h->base + bb.xin_cls, (long)D * 4, B, D * 4);
    proj_in = h->base + bb.o_cls;
    proj_res = h->base + bb.xin_cls;
    Ma = B;
    Mf = B;
  }
  GemmEpilogue e2;
  e2.bias = (const float*)h->wb(l, "attn.proj.bias");
  e2.residual = proj_res;
  void* xp_dst = h->base + (shrinks ? bb.xp_full : bb.xp);
  gemm(c, proj_in, D, 1, h->wb(l, "attn.proj.weight"), D, 1, xp_dst, 1, Ma, D, D, e2);
  if (is_drop) {
    int M = Ta - 1;
    token_select(c.stream, h->at<float>(bb.p), B, H, M, k, h->at<float>(bb.s), h->at<int>(bb.kept), h->at<int>(bb.dropped));
    if (kept_out != nullptr)
      cudaMemcpyAsync(kept_out, h->base + bb.kept, (size_t)B * k * sizeof(int), cudaMemcpyDeviceToDevice, c.stream);
    if (shrinks)
      gather_fuse(cf, h->base + bb.xp_full, B, M, D, k, h->at<int>(bb.kept), h->at<int>(bb.dropped), h->at<float>(bb.s),
                  h->cfg.fuse_mode, h->base + bb.xp);
  }
  if (fp8 && !is_moe(h, l)) {
    layernorm_fwd_e4m3(c, h->at<float>(bb.xp), D, (const float*)h->wb(l, "norm2.weight"), (const float*)h->wb(l, "norm2.bias"),
                       h->base + h->off_yq, h->at<float>(h->off_yq_s), Mf, D, d.ln_eps);
    GemmEpilogue q3;
    q3.bias = (const float*)h->wb(l, "mlp.fc1.bias");
    q3.act = 1;
    if (gemm_tc_e4m3(c, h->base + h->off_yq, h->at<float>(h->off_yq_s), h->base + h->q_fc1[l], h->at<float>(h->q_fc1_s[l]),
                     h->base + bb.hh, Mf, F, D, q3) != 0)
      return set_err(h->err, BSR_ERR_CUDA, "8-bit GEMM set-up failed");
    GemmEpilogue q4;
    q4.bias = (const float*)h->wb(l, "mlp.fc2.bias");
    q4.residual = h->base + bb.xp;
    gemm(c, h->base + bb.hh, F, 1, h->wb(l, "mlp.fc2.weight"), F, 1, h->base + bb.x_out, 1, Mf, D, F, q4);
    return BSR_OK;
  }
  layernorm_fwd(c, h->at<float>(bb.xp), D, (const float*)h->wb(l, "norm2.weight"), (const float*)h->wb(l, "norm2.bias"),
                h->base + bb.y2, 0, save ? h->at<float>(bb.mean2) : nullptr, save ? h->at<float>(bb.rstd2) : nullptr, Mf, D, d.ln_eps);
  if (is_moe(h, l)) {
    // MoE layer in place of the FFN (Section 5.2): route, run the chosen experts as grouped GEMMs, combine
    int E = d.moe_experts, K = d.moe_top_k;
    MoeBufs mb = moe_bufs(h, bb);
    int cap = moe_rows_cap(Mf, E, K);
    // Gate logits of every task at once as one product y Wg^T ([Mf, D] x [D, tasks E]) on the tensor cores; they land in
    // the expert-output buffer, which is not written before the routing has consumed them.  (Small or odd gate shapes:
    // the routing kernel forms the logits itself.)
    int NG = d.num_tasks * E;
    const float* logits = nullptr;
    if (c.use_tc && d.dtype == BSR_DTYPE_BF16 && Mf >= 256 && NG % 8 == 0 && (size_t)Mf * NG <= (size_t)cap * D) {
      GemmEpilogue none;
      gemm(c, h->base + bb.y2, D, 1, h->wb(l, "moe.gate.weight"), D, 1, mb.og, 1, Mf, NG, D, none);
      logits = mb.og;
    }
    moe_route(c, mb, h->base + bb.y2, h->wb(l, "moe.gate.weight"), task_ids, tail ? 1 : Tf, Mf, D, E, K, d.num_tasks, logits, NG);
    GemmEpilogue m1;
    m1.bias = (const float*)h->wb(l, "moe.fc1.bias");
    m1.act = 1;
    m1.aux_out = save ? mb.zg : nullptr;
    int rc1 = gemm_tc_grouped_rows(c, mb.xg, h->wb(l, "moe.fc1.weight"), 0, mb.hg, 0, cap, F, D, E, mb.tile_expert, m1);
    GemmEpilogue m2;
    m2.bias = (const float*)h->wb(l, "moe.fc2.bias");
    int rc2 = gemm_tc_grouped_rows(c, mb.hg, h->wb(l, "moe.fc2.weight"), 0, mb.og, 1, cap, D, F, E, mb.tile_expert, m2);
    if (rc1 != 0 || rc2 != 0) return set_err(h->err, BSR_ERR_CUDA, "grouped GEMM set-up failed (%d, %d)", rc1, rc2);
    moe_combine(c, mb, h->at<float>(bb.xp), h->at<float>(bb.x_out), Mf, D, K);
    return BSR_OK;
  }
  GemmEpilogue e3;
  e3.bias = (const float*)h->wb(l, "mlp.fc1.bias");
  e3.act = 1;
  e3.aux_out = save ? h->base + bb.z : nullptr;
  gemm(c, h->base + bb.y2, D, 1, h->wb(l, "mlp.fc1.weight"), D, 1, h->base + bb.hh, 0, Mf, F, D, e3);
  GemmEpilogue e4;
  e4.bias = (const float*)h->wb(l, "mlp.fc2.bias");
  e4.residual = h->base + bb.xp;
  gemm(c, h->base + bb.hh, F, 1, h->wb(l, "mlp.fc2.weight"), F, 1, h->base + bb.x_out, 1, Mf, D, F, e4);
  return BSR_OK;
}

// Backward of one trainable block (Eq. 2-5).  dxo: gradient at the block output [B*Tf, D]; dxi receives the
// gradient at the block input unless it is null (earliest trainable block: Eq. 8, nothing flows further).
struct GradStream {      // gradient of the residual stream: float rows, plus the bf16 copy the GEMMs read (bf16 only)
  float* f;
  void* c;
};

int block_backward(bsr_handle* h, const Ctx& c, int l, int B, GradStream dxo, GradStream dxi, bool need_dxi, const int* task_ids) {
  const bsr_dims& d = h->cfg.dims;
  const Schedule& s = h->sched;
  const BlockBufs& bb = h->bufs_train[l];
  int D = d.dim, F = d.mlp_hidden, H = d.heads, hd = D / H;
  int Ta = s.ta[l], Tf = s.tf[l], k = s.k[l];
  int Ma = B * Ta, Mf = B * Tf;
  bool shrinks = k >= 0 && Tf != Ta;
  bool bf = d.dtype == BSR_DTYPE_BF16;
  bool tail = cls_tail(h, l);
  bool pg = (h->cfg.trainable_mask >> l) & 1u;     // a frozen block inside the gradient path only passes gradients on (Eq. 2)
  size_t es = dtype_size(d.dtype);
  int Mdense = Ma;
  if (tail) { Ma = B; Mf = B; }          // FFN and projection gradients live on the classification rows only
  Ctx cf = c;
  cf.dtype = 0;
  float* csp = h->at<float>(h->off_cs_partials);
  float* lnp = h->at<float>(h->off_ln_partials);
  void* dz = h->base + h->off_dz;
  void* dy = h->base + h->off_dy;
  GradStream dxg = {h->at<float>(h->off_dxg), bf ? (void*)(h->base + h->off_dxg_c) : nullptr};
  GradStream dxp = shrinks ? GradStream{h->at<float>(h->off_dxp), bf ? (void*)(h->base + h->off_dxp_c) : nullptr} : dxg;
  void* d_o = h->base + h->off_do;
  void* dqkv = h->base + h->off_dqkv;
  auto op = [&](const GradStream& g) -> const void* { return bf ? g.c : (const void*)g.f; };   // GEMM operand view
  GemmEpilogue none;
  if (is_moe(h, l)) {
    int E = d.moe_experts, K = d.moe_top_k;
    MoeBufs mb = moe_bufs(h, bb);
    int cap = moe_rows_cap(Mf, E, K);
    void* dog = h->base + h->off_m_dog;
    void* dzg = h->base + h->off_m_dzg;
    void* dxg = h->base + h->off_m_dxg;
    float* dwsel = h->at<float>(h->off_m_dw);
    moe_combine_bwd(c, mb, dxo.f, dog, dwsel, Mf, D, E, K);
    GemmEpilogue eg;
    eg.act = 2;
    eg.aux_in = mb.zg;
    int r1 = gemm_tc_grouped_rows(c, dog, h->wb(l, "moe.fc2.weight"), 1, dzg, 0, cap, F, D, E, mb.tile_expert, eg);
    int r2 = 0, r4 = 0;
    if (pg) {
      r2 = gemm_tc_grouped_wgrad(c, dog, mb.hg, h->gb(l, "moe.fc2.weight"), cap, D, F, E, mb.seg_start);
      moe_seg_colsum(c, mb, dog, D, E, h->gb(l, "moe.fc2.bias"));
    }
    int r3 = gemm_tc_grouped_rows(c, dzg, h->wb(l, "moe.fc1.weight"), 1, dxg, 0, cap, D, F, E, mb.tile_expert, none);
    if (pg) {
      r4 = gemm_tc_grouped_wgrad(c, dzg, mb.xg, h->gb(l, "moe.fc1.weight"), cap, F, D, E, mb.seg_start);
      moe_seg_colsum(c, mb, dzg, F, E, h->gb(l, "moe.fc1.bias"));
    }
    if (r1 || r2 || r3 || r4) return set_err(h->err, BSR_ERR_CUDA, "grouped GEMM set-up failed (%d, %d, %d, %d)", r1, r2, r3, r4);
    moe_gate_bwd(c, mb, dxg, dwsel, h->wb(l, "moe.gate.weight"), task_ids, tail ? 1 : Tf, d.num_tasks, Mf, D, E, K, dy,
                 h->at<float>(h->off_m_dsel), pg ? h->gb(l, "moe.gate.weight") : nullptr);
  } else {
  // FFN second layer: dz = (dxo W2) * GELU'(z); dW2 = dxo^T h; db2 = column sums of dxo
  GemmEpilogue eg;
  eg.act = 2;
  eg.aux_in = h->base + bb.z;
  if (pg) eg.aux_out = h->base + bb.hh;       // GELU(z) again, into scratch, for the weight gradient below
  gemm(c, op(dxo), D, 1, h->wb(l, "mlp.fc2.weight"), 1, F, dz, 0, Mf, F, D, eg);
  if (pg) {
    gemm(c, op(dxo), 1, D, h->base + bb.hh, 1, F, h->gb(l, "mlp.fc2.weight"), 1, D, F, Mf, none);
    // db2 = column sums of dxo: they came out of the following block's LayerNorm backward, which wrote dxo
    if (l == d.depth - 1) colsum(cf, dxo.f, Mf, D, csp, h->gb(l, "mlp.fc2.bias"));
  }
  // FFN first layer
  gemm(c, dz, F, 1, h->wb(l, "mlp.fc1.weight"), 1, D, dy, 0, Mf, D, F, none);
  if (pg) {
    gemm(c, dz, 1, F, h->base + bb.y2, 1, D, h->gb(l, "mlp.fc1.weight"), 1, F, D, Mf, none);
    colsum(c, dz, Mf, F, csp, h->gb(l, "mlp.fc1.bias"));
  }
  }
  layernorm_bwd(c, dy, 0, h->at<float>(bb.xp), D, h->at<float>(bb.mean2), h->at<float>(bb.rstd2),
                (const float*)h->wb(l, "norm2.weight"), dxo.f, dxg.f, D, shrinks ? nullptr : dxg.c, lnp,
                pg ? h->gb(l, "norm2.weight") : nullptr, pg ? h->gb(l, "norm2.bias") : nullptr, Mf, D,
                (pg && !shrinks) ? h->gb(l, "attn.proj.bias") : nullptr);   // dx' = dxg here: its column sums are the projection's bias gradient
  const float* cls_extra = nullptr;
  if (shrinks) {
    gather_fuse_bwd(c, dxg.f, h->base + bb.xp_full, B, Ta - 1, D, k, h->at<int>(bb.kept), h->at<int>(bb.dropped),
                    h->at<float>(bb.s), h->cfg.fuse_mode, dxp.f, dxp.c, h->at<float>(h->off_escore), h->base + bb.xp);
    if (h->cfg.fuse_mode != BSR_FUSE_NONE) cls_extra = h->at<float>(h->off_escore);
  }
  // attention output projection
  bool tail_cls_attn = false;
  const float* ln1_res = dxp.f;
  if (!tail) {
    gemm(c, op(dxp), D, 1, h->wb(l, "attn.proj.weight"), 1, D, d_o, 0, Ma, D, D, none);
    if (pg) {
      gemm(c, op(dxp), 1, D, h->base + bb.o, 1, D, h->gb(l, "attn.proj.weight"), 1, D, D, Ma, none);
      if (shrinks) colsum(cf, dxp.f, Ma, D, csp, h->gb(l, "attn.proj.bias"));
    }
  } else {
    // B rows: dO_cls = dx'_cls Wo, dWo = dx'_cls^T o_cls; then both gradients go back into zeroed dense tensors
    void* do_cls = h->base + h->off_dy;                      // free at this point
    gemm(c, op(dxp), D, 1, h->wb(l, "attn.proj.weight"), 1, D, do_cls, 0, B, D, D, none);
    if (pg) {
      gemm(c, op(dxp), 1, D, h->base + bb.o_cls, 1, D, h->gb(l, "attn.proj.weight"), 1, D, D, B, none);
      if (shrinks) colsum(cf, dxp.f, B, D, csp, h->gb(l, "attn.proj.bias"));
    }
    // with the classification-row attention, dqkv comes straight from do_cls; otherwise dO is scattered into a zeroed
    // dense tensor for the general kernel
    tail_cls_attn = attention_cls_bwd(c, h->base + bb.qkv, do_cls, dqkv, B, Ta, H, hd) == 0;
    if (!tail_cls_attn) {
      cudaMemsetAsync(d_o, 0, (size_t)Mdense * D * es, c.stream);
      copy_rows(c.stream, do_cls, (long)D * es, d_o, (long)Ta * D * es, B, (int)(D * es));
    }
    float* dense_res = h->at<float>(h->off_dxp);
    cudaMemsetAsync(dense_res, 0, (size_t)Mdense * D * 4, c.stream);
    copy_rows(c.stream, dxp.f, (long)D * 4, dense_res, (long)Ta * D * 4, B, D * 4);
    ln1_res = dense_res;
    Ma = Mdense;
  }
  // the gradient this block hands to block l-1 is that block's output gradient: its column sums are the bias gradient
  // of block l-1's second FFN layer (dense FFN, trainable)
  float* prev_fc2_bias = (need_dxi && l > 0 && ((h->cfg.trainable_mask >> (l - 1)) & 1u) && !is_moe(h, l - 1)) ? h->gb(l - 1, "mlp.fc2.bias") : nullptr;
  if (!tail_cls_attn) {
    int rc = attention_bwd(c, h->base + bb.qkv, h->base + bb.o, d_o, h->at<float>(bb.lse), h->at<float>(h->off_delta),
                           cls_extra, dqkv, B, Ta, H, hd);
    if (rc != 0) return set_err(h->err, BSR_ERR_UNSUPPORTED, "attention backward: %d tokens do not fit this kernel", Ta);
  }
  // QKV projection
  gemm(c, dqkv, 3 * D, 1, h->wb(l, "attn.qkv.weight"), 1, D, dy, 0, Ma, D, 3 * D, none);
  if (pg) {
    gemm(c, dqkv, 1, 3 * D, h->base + bb.y1, 1, D, h->gb(l, "attn.qkv.weight"), 1, 3 * D, D, Ma, none);
    colsum(c, dqkv, Ma, 3 * D, csp, h->gb(l, "attn.qkv.bias"));
  }
  layernorm_bwd(c, dy, 0, h->at<float>(bb.x_in), D, h->at<float>(bb.mean1), h->at<float>(bb.rstd1),
                (const float*)h->wb(l, "norm1.weight"), ln1_res, need_dxi ? dxi.f : nullptr, D, need_dxi ? dxi.c : nullptr, lnp,
                pg ? h->gb(l, "norm1.weight") : nullptr, pg ? h->gb(l, "norm1.bias") : nullptr, Ma, D, prev_fc2_bias);
  return BSR_OK;
}

HeadDesc head_desc(bsr_handle* h) {
  const bsr_dims& d = h->cfg.dims;
  HeadDesc hd;
  memset(&hd, 0, sizeof(hd));
  hd.num_tasks = d.num_tasks;
  hd.D = d.dim;
  for (int t = 0; t < d.num_tasks; ++t) {
    std::string n = "head." + std::to_string(t);
    hd.ncls[t] = d.num_classes[t];
    hd.cmax = d.num_classes[t] > hd.cmax ? d.num_classes[t] : hd.cmax;
    hd.w[t] = h->w((n + ".weight").c_str());
    hd.bias[t] = (const float*)h->w((n + ".bias").c_str());
    hd.dw[t] = h->gradp(n + ".weight");
    hd.db[t] = h->gradp(n + ".bias");
  }
  return hd;
}

// Forward through all blocks.  train: blocks >= t0 write the activation arena.  Returns the offset of the last output.
int forward_all(bsr_handle* h, const Ctx& c, const void* images, int B, bool train, size_t* x_last_off, const int* task_ids,
                const long long* img_offset = nullptr) {
  const bsr_dims& d = h->cfg.dims;
  int D = d.dim;
  int g = d.image_size / d.patch_size, N = g * g;
  int pin = d.in_chans * d.patch_size * d.patch_size;
  patchify(c, images, h->base + h->off_patches, B, d.in_chans, d.image_size, d.patch_size, img_offset);
  GemmEpilogue ep;
  ep.bias = (const float*)h->w("patch_embed.bias");
  gemm(c, h->base + h->off_patches, pin, 1, h->w("patch_embed.weight"), pin, 1, h->base + h->off_emb, 0, B * N, D, pin, ep);
  int first_train = train ? h->t0 : d.depth;
  size_t x0 = (first_train == 0) ? h->bufs_train[0].x_in : h->bufs_frozen[0].x_in;
  assemble_tokens(c, h->base + h->off_emb, (const float*)h->w("cls_token"), (const float*)h->w("pos_embed"), h->at<float>(x0), B, N, D);
  int* kept_all = h->at<int>(h->off_kept_all);
  size_t kept_off = 0;
  size_t cur = x0;
  for (int l = 0; l < d.depth; ++l) {
    BlockBufs bb;
    bool save = l >= first_train;
    if (save) {
      bb = h->bufs_train[l];
    } else {
      bb = h->bufs_frozen[l & 1];
      if (l + 1 == first_train && first_train < d.depth) bb.x_out = h->bufs_train[l + 1].x_in;   // hand over to the first trainable block
    }
    bb.x_in = cur;
    if (is_moe(h, l)) { bb.m_eidx = h->moe_rec_eidx[l]; bb.m_ew = h->moe_rec_ew[l]; }
    if (h->sched.k[l] >= 0) bb.s = h->score_rec[l];
    int* kept_dst = nullptr;
    if (h->sched.k[l] >= 0) { kept_dst = kept_all + kept_off; kept_off += (size_t)B * h->sched.k[l]; }
    int rc = block_forward(h, c, l, B, bb, save, kept_dst, task_ids);
    if (rc != BSR_OK) return rc;
    cur = bb.x_out;
  }
  *x_last_off = cur;
  return BSR_OK;
}

size_t kept_total(const bsr_handle* h, int B) {
  size_t n = 0;
  for (int l = 0; l < h->cfg.dims.depth; ++l)
    if (h->sched.k[l] >= 0) n += (size_t)B * h->sched.k[l];
  return n;
}

int check_batch(bsr_handle* h, const void* images, int batch) {
  if (h == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "handle is null");
  if (images == nullptr) return set_err(h->err, BSR_ERR_INVALID_ARG, "images_dev is null");
  if (batch < 1 || batch > h->cfg.max_batch) return set_err(h->err, BSR_ERR_INVALID_ARG, "batch %d outside [1, %d]", batch, h->cfg.max_batch);
  return BSR_OK;
}

}  // namespace

// =================================================================================================
// C ABI
// =================================================================================================
extern "C" {

int32_t bsr_token_schedule(const bsr_config* cfg, int32_t* ta, int32_t* tf, int32_t* keep) {
  if (cfg == nullptr || ta == nullptr || tf == nullptr || keep == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "null argument");
  Schedule s;
  int rc = compute_schedule(cfg, &s, g_error);
  if (rc != BSR_OK) return rc;
  for (int l = 0; l < cfg->dims.depth; ++l) { ta[l] = s.ta[l]; tf[l] = s.tf[l]; keep[l] = s.k[l]; }
  return BSR_OK;
}

int32_t bsr_workspace_bytes(const bsr_config* cfg, size_t* bytes) {
  if (bytes == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "bytes is null");
  int rc = validate(cfg, g_error);
  if (rc != BSR_OK) return rc;
  bsr_handle tmp;
  tmp.cfg = *cfg;
  compute_schedule(cfg, &tmp.sched, g_error);
  build_tensors(&tmp);
  *bytes = plan(&tmp);
  return BSR_OK;
}

int32_t bsr_create(const bsr_config* cfg, void* workspace, size_t bytes, bsr_handle** out) {
  if (out == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "out is null");
  *out = nullptr;
  int rc = validate(cfg, g_error);
  if (rc != BSR_OK) return rc;
  if (workspace == nullptr || ((uintptr_t)workspace & 255) != 0) return set_err(g_error, BSR_ERR_INVALID_ARG, "workspace must be non-null and 256-byte aligned");
  bsr_handle* h = new bsr_handle();
  h->cfg = *cfg;
  snprintf(h->err, sizeof(h->err), "no error");
  compute_schedule(cfg, &h->sched, h->err);
  build_tensors(h);
  size_t need = plan(h);
  if (bytes < need) {
    delete h;
    return set_err(g_error, BSR_ERR_WORKSPACE_TOO_SMALL, "workspace of %zu bytes given, %zu needed", bytes, need);
  }
  h->base = (char*)workspace;
  h->bytes = bytes;
  h->lr = cfg->lr;
  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
    delete h;
    return set_err(g_error, BSR_ERR_CUDA, "no usable CUDA device: %s", cudaGetErrorString(cudaGetLastError()));
  }
  h->sm_count = prop.multiProcessorCount;
  if (prop.major != 10) {
    delete h;
    return set_err(g_error, BSR_ERR_UNSUPPORTED, "this library is built for sm_100a only (device is sm_%d%d)", prop.major, prop.minor);
  }
  // optimiser state and status start at zero; the chunk table is uploaded once
  cudaMemsetAsync(h->base + h->off_status, 0, 256, 0);
  cudaMemsetAsync(h->base + h->off_m, 0, h->n_flat * 4, 0);
  cudaMemsetAsync(h->base + h->off_v, 0, h->n_flat * 4, 0);
  cudaMemsetAsync(h->base + h->off_grad, 0, h->n_flat * 4, 0);
  cudaMemsetAsync(h->base + h->off_master, 0, h->n_flat * 4, 0);
  std::vector<AdamChunk> chunks;
  for (auto& t : h->tensors) {
    if (!t.trainable) continue;
    bool has_shadow = t.matrix && cfg->dims.dtype == BSR_DTYPE_BF16;
    for (size_t o = 0; o < t.numel; o += ADAM_CHUNK) {
      AdamChunk ch;
      ch.offset = (uint32_t)(t.flat + o);
      ch.count = (uint32_t)((t.numel - o) < ADAM_CHUNK ? (t.numel - o) : ADAM_CHUNK);
      ch.shadow = has_shadow ? (int64_t)((t.w_off - h->off_weights) / 2 + o) : -1;
      ch.decay = t.decay ? 1u : 0u;
      ch.pad = 0;
      chunks.push_back(ch);
    }
  }
  if (!chunks.empty())
    cudaMemcpy(h->base + h->off_chunks, chunks.data(), chunks.size() * sizeof(AdamChunk), cudaMemcpyHostToDevice);
  if (!h->guards.empty()) {
    std::vector<unsigned long long> table(h->guards.begin(), h->guards.end());
    cudaMemcpy(h->base + h->off_guard_table, table.data(), table.size() * sizeof(unsigned long long), cudaMemcpyHostToDevice);
    guards_write(0, h->base, h->at<unsigned long long>(h->off_guard_table), (int)table.size(), (int)(GUARD_BYTES / 4), GUARD_WORD);
  }
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    delete h;
    return set_err(g_error, BSR_ERR_CUDA, "workspace initialisation failed: %s", cudaGetErrorString(e));
  }
  // host objects of the side lane (no device memory); without them the reductions simply stay on the main stream
  bool lane = cudaStreamCreateWithFlags(&h->side.stream, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&h->side.fork, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; i < 3 && lane; ++i) lane = cudaEventCreateWithFlags(&h->side.done[i], cudaEventDisableTiming) == cudaSuccess;
  if (!lane) { cudaGetLastError(); h->side.stream = nullptr; }
  *out = h;
  return BSR_OK;
}

int32_t bsr_destroy(bsr_handle* h) {
  if (h != nullptr) {
    for (cudaEvent_t ev : h->prof.events) cudaEventDestroy(ev);
    for (auto& g : h->graphs) cudaGraphExecDestroy(g.exec);
    for (int i = 0; i < 2; ++i) {
      if (h->ev_copied[i]) cudaEventDestroy(h->ev_copied[i]);
      if (h->ev_done[i]) cudaEventDestroy(h->ev_done[i]);
    }
    if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
    if (h->side.fork) cudaEventDestroy(h->side.fork);
    for (int i = 0; i < 3; ++i)
      if (h->side.done[i]) cudaEventDestroy(h->side.done[i]);
    if (h->side.stream) cudaStreamDestroy(h->side.stream);
  }
  delete h;
  return BSR_OK;
}

const char* bsr_last_error(const bsr_handle* h) { return h ? h->err : g_error; }

int32_t bsr_set_param(bsr_handle* h, const char* name, const void* src, size_t count, int32_t src_dtype, int32_t src_is_device,
                      void* stream) {
  if (h == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "handle is null");
  if (name == nullptr || src == nullptr) return set_err(h->err, BSR_ERR_INVALID_ARG, "null argument");
  if (src_dtype != BSR_DTYPE_FP32 && src_dtype != BSR_DTYPE_BF16) return set_err(h->err, BSR_ERR_INVALID_ARG, "src_dtype must be fp32 (0) or bf16 (1)");
  auto it = h->index.find(name);
  if (it == h->index.end()) return set_err(h->err, BSR_ERR_INVALID_ARG, "unknown parameter '%s'", name);
  const Tensor& t = h->tensors[it->second];
  if (count != t.numel) return set_err(h->err, BSR_ERR_INVALID_ARG, "'%s' has %zu elements, %zu given", name, t.numel, count);
  Ctx c = make_ctx(h, stream);
  Ctx cs = c;                       // conversions from the source's type
  cs.dtype = src_dtype;
  size_t es_src = dtype_size(src_dtype);
  if (!src_is_device) {             // host source: through the staging area (sized for the largest tensor as float)
    cudaMemcpyAsync(h->base + h->off_stage, src, count * es_src, cudaMemcpyHostToDevice, c.stream);
    src = h->base + h->off_stage;
  }
  auto to_float = [&](float* dst) {
    if (src_dtype == BSR_DTYPE_FP32) cudaMemcpyAsync(dst, src, count * 4, cudaMemcpyDeviceToDevice, c.stream);
    else convert_to_float(cs, src, dst, count);
  };
  if (t.trainable) to_float(h->at<float>(h->off_master) + t.flat);
  bool alias_master = t.trainable && (!t.matrix || c.dtype == BSR_DTYPE_FP32);
  if (!alias_master) {
    if (!t.matrix || c.dtype == BSR_DTYPE_FP32) to_float(h->at<float>(t.w_off));
    else if (src_dtype == BSR_DTYPE_BF16) cudaMemcpyAsync(h->base + t.w_off, src, count * 2, cudaMemcpyDeviceToDevice, c.stream);
    else convert_from_float(c, (const float*)src, h->base + t.w_off, count);
  }
  if (h->cfg.frozen_fp8 && t.matrix && !t.trainable && t.name.rfind("blocks.", 0) == 0) {     // 8-bit copy of a prefix weight
    int l = atoi(t.name.c_str() + 7);
    int D = h->cfg.dims.dim, F = h->cfg.dims.mlp_hidden;
    bool qkv = t.name.find(".attn.qkv.weight") != std::string::npos, fc1 = t.name.find(".mlp.fc1.weight") != std::string::npos;
    if (l < h->t0 && h->q_qkv[l] != 0 && (qkv || fc1))
      quantize_rows_e4m3(c, h->base + t.w_off, qkv ? 3 * D : F, D, h->base + (qkv ? h->q_qkv[l] : h->q_fc1[l]),
                         h->at<float>(qkv ? h->q_qkv_s[l] : h->q_fc1_s[l]));
  }
  return check_cuda(h, "bsr_set_param");
}

int32_t bsr_get_tensor(bsr_handle* h, const char* name, float* dst, size_t count, void* stream) {
  if (h == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "handle is null");
  if (name == nullptr || dst == nullptr) return set_err(h->err, BSR_ERR_INVALID_ARG, "null argument");
  Ctx c = make_ctx(h, stream);
  std::string n(name);
  const float* src = nullptr;
  size_t numel = 0;
  if (n == "loss") { src = h->at<float>(h->off_loss); numel = 1; }
  else if (n == "logits") {
    int cmax = 0;
    for (int t = 0; t < h->cfg.dims.num_tasks; ++t) cmax = h->cfg.dims.num_classes[t] > cmax ? h->cfg.dims.num_classes[t] : cmax;
    src = h->at<float>(h->off_logits); numel = (size_t)h->cfg.max_batch * cmax;
  } else if (n.rfind("moe_experts/", 0) == 0) {
    int l = atoi(n.c_str() + 12);
    if (l < 0 || l >= h->cfg.dims.depth || !is_moe(h, l)) return set_err(h->err, BSR_ERR_INVALID_ARG, "'%s': not an MoE block", name);
    size_t recorded = (size_t)h->cfg.max_batch * h->sched.tf[l] * h->cfg.dims.moe_top_k;
    if (count < 1 || count > recorded) return set_err(h->err, BSR_ERR_INVALID_ARG, "'%s' records at most %zu values, %zu asked for", name, recorded, count);
    convert_int_to_float(c.stream, h->at<int>(h->moe_rec_eidx[l]), dst, count);
    return check_cuda(h, "bsr_get_tensor");
  } else if (n.rfind("fp8/", 0) == 0) {
    // the E4M3 copy of a prefix weight, scaled back to float: "fp8/blocks.<l>.attn.qkv.weight" or "...mlp.fc1.weight"
    std::string pn = n.substr(4);
    auto it = h->index.find(pn);
    int l = pn.rfind("blocks.", 0) == 0 ? atoi(pn.c_str() + 7) : -1;
    bool qkv = pn.find(".attn.qkv.weight") != std::string::npos, fc1 = pn.find(".mlp.fc1.weight") != std::string::npos;
    if (it == h->index.end() || l < 0 || l >= h->cfg.dims.depth || !(qkv || fc1) || h->q_qkv[l] == 0)
      return set_err(h->err, BSR_ERR_INVALID_ARG, "'%s' has no 8-bit copy", name);
    int rows = qkv ? 3 * h->cfg.dims.dim : h->cfg.dims.mlp_hidden, cols = h->cfg.dims.dim;
    if (count != (size_t)rows * cols) return set_err(h->err, BSR_ERR_INVALID_ARG, "'%s' has %zu elements, %zu given", name, (size_t)rows * cols, count);
    dequantize_rows_e4m3(c, h->base + (qkv ? h->q_qkv[l] : h->q_fc1[l]), h->at<float>(qkv ? h->q_qkv_s[l] : h->q_fc1_s[l]), rows, cols, dst);
    return check_cuda(h, "bsr_get_tensor");
  } else if (n.rfind("scores/", 0) == 0) {
    int l = atoi(n.c_str() + 7);
    if (l < 0 || l >= h->cfg.dims.depth || h->sched.k[l] < 0) return set_err(h->err, BSR_ERR_INVALID_ARG, "'%s': not a token drop location", name);
    src = h->at<float>(h->score_rec[l]); numel = (size_t)h->cfg.max_batch * (h->sched.ta[l] - 1);
  } else {
    size_t base_off = 0;
    std::string pn = n;
    bool state = false;
    if (n.rfind("grad/", 0) == 0) { base_off = h->off_grad; pn = n.substr(5); state = true; }
    else if (n.rfind("adam_m/", 0) == 0) { base_off = h->off_m; pn = n.substr(7); state = true; }
    else if (n.rfind("adam_v/", 0) == 0) { base_off = h->off_v; pn = n.substr(7); state = true; }
    auto it = h->index.find(pn);
    if (it == h->index.end()) return set_err(h->err, BSR_ERR_INVALID_ARG, "unknown tensor '%s'", name);
    const Tensor& t = h->tensors[it->second];
    numel = t.numel;
    if (state) {
      if (!t.trainable) return set_err(h->err, BSR_ERR_INVALID_ARG, "'%s' is frozen: it has no gradient or optimiser state", pn.c_str());
      src = h->at<float>(base_off) + t.flat;
    } else if (t.trainable) {
      src = h->at<float>(h->off_master) + t.flat;
    } else if (!t.matrix) {
      src = h->at<float>(t.w_off);
    } else {
      if (count != numel) return set_err(h->err, BSR_ERR_INVALID_ARG, "'%s' has %zu elements, %zu given", name, numel, count);
      convert_to_float(c, h->base + t.w_off, dst, numel);
      return check_cuda(h, "bsr_get_tensor");
    }
  }
  if (count != numel) return set_err(h->err, BSR_ERR_INVALID_ARG, "'%s' has %zu elements, %zu given", name, numel, count);
  cudaMemcpyAsync(dst, src, numel * 4, cudaMemcpyDeviceToDevice, c.stream);
  return check_cuda(h, "bsr_get_tensor");
}

int32_t bsr_set_lr(bsr_handle* h, float lr) {
  if (h == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "handle is null");
  h->lr = lr;
  return BSR_OK;
}

int32_t bsr_set_step(bsr_handle* h, int64_t steps_done) {
  if (h == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "handle is null");
  if (steps_done < 0) return set_err(h->err, BSR_ERR_INVALID_ARG, "steps_done must not be negative");
  h->step = steps_done;
  return BSR_OK;
}

// Enqueues every kernel of one step on `stream` (forward, loss, backward, AdamW reading its scalars from device memory).
// loss_out may be null (the multi-step loop writes the loss itself); img_offset as in forward_all.
static void enqueue_optimizer(bsr_handle* h, const Ctx& c);
static int enqueue_train_step(bsr_handle* h, const void* images, const int32_t* labels, const int32_t* task_ids, int32_t batch,
                              void* stream, float* loss_out, int32_t* kept_out, const long long* img_offset = nullptr,
                              bool with_update = true) {
  int rc;
  const bsr_dims& d = h->cfg.dims;
  Ctx c = make_ctx(h, stream);
  int D = d.dim, B = batch;
  size_t es = dtype_size(d.dtype);
  size_t x_last = 0;
  rc = forward_all(h, c, images, B, true, &x_last, task_ids, img_offset);
  if (rc != BSR_OK) return rc;
  int Tl = cls_tail(h, d.depth - 1) ? 1 : h->sched.tf[d.depth - 1];   // rows per image in the last block's output
  HeadDesc hd = head_desc(h);
  float* xn = h->at<float>(h->off_xn);
  layernorm_fwd(c, h->at<float>(x_last), (long)Tl * D, (const float*)h->w("norm.weight"), (const float*)h->w("norm.bias"), xn, 1,
                h->at<float>(h->off_meanf), h->at<float>(h->off_rstdf), B, D, d.ln_eps);
  head_fwd(c, hd, xn, task_ids, h->at<float>(h->off_logits), B);
  cross_entropy(c, hd, h->at<float>(h->off_logits), labels, task_ids, h->at<float>(h->off_per_image), h->at<float>(h->off_dlogits),
                h->at<float>(h->off_loss), B);
  if (loss_out != nullptr) cudaMemcpyAsync(loss_out, h->at<float>(h->off_loss), 4, cudaMemcpyDeviceToDevice, c.stream);
  if (kept_out != nullptr && kept_total(h, B) > 0)
    cudaMemcpyAsync(kept_out, h->base + h->off_kept_all, kept_total(h, B) * 4, cudaMemcpyDeviceToDevice, c.stream);
  // backward: head, final LayerNorm, trainable blocks in reverse, nothing before the earliest one
  head_bwd(c, hd, xn, h->at<float>(h->off_dlogits), task_ids, h->at<float>(h->off_dxn), B);
  float* lnp = h->at<float>(h->off_ln_partials);
  bool bf = d.dtype == BSR_DTYPE_BF16;
  if (h->t0 < d.depth) {
    GradStream dxo = {h->at<float>(h->off_dxa), bf ? (void*)(h->base + h->off_dxa_c) : nullptr};
    GradStream dxi = {h->at<float>(h->off_dxb), bf ? (void*)(h->base + h->off_dxb_c) : nullptr};
    // only the classification rows of the last block's output receive a gradient
    cudaMemsetAsync(dxo.f, 0, (size_t)B * Tl * D * 4, c.stream);
    if (bf) cudaMemsetAsync(dxo.c, 0, (size_t)B * Tl * D * es, c.stream);
    layernorm_bwd(c, h->at<float>(h->off_dxn), 1, h->at<float>(x_last), (long)Tl * D, h->at<float>(h->off_meanf), h->at<float>(h->off_rstdf),
                  (const float*)h->w("norm.weight"), nullptr, dxo.f, (long)Tl * D, dxo.c, lnp, h->gradp("norm.weight"), h->gradp("norm.bias"), B, D);
    for (int l = d.depth - 1; l >= h->t0; --l) {
      rc = block_backward(h, c, l, B, dxo, dxi, l > h->t0, task_ids);
      if (rc != BSR_OK) return rc;
      GradStream t = dxo; dxo = dxi; dxi = t;
    }
  } else {
    layernorm_bwd(c, h->at<float>(h->off_dxn), 1, h->at<float>(x_last), (long)Tl * D, h->at<float>(h->off_meanf), h->at<float>(h->off_rstdf),
                  (const float*)h->w("norm.weight"), nullptr, nullptr, 0, nullptr, lnp, h->gradp("norm.weight"), h->gradp("norm.bias"), B, D);
  }
  side_join_all(c);                      // every gradient is complete on the main stream from here on
  if (with_update) enqueue_optimizer(h, c);
  return BSR_OK;
}

// The update of the trainable parameters from the flat gradient buffer; learning rate and bias corrections are read
// from device memory (the three scalars at status + 128).
static void enqueue_optimizer(bsr_handle* h, const Ctx& c) {
  if (h->cfg.optimizer == BSR_OPT_SGD)
    sgd_momentum(c, h->at<AdamChunk>(h->off_chunks), h->n_chunks, h->at<float>(h->off_master), h->at<float>(h->off_grad),
                 h->at<float>(h->off_m), h->base + h->off_weights, h->at<float>(h->off_status + 128), h->cfg.momentum, h->cfg.weight_decay);
  else
    adamw(c, h->at<AdamChunk>(h->off_chunks), h->n_chunks, h->at<float>(h->off_master), h->at<float>(h->off_grad), h->at<float>(h->off_m),
          h->at<float>(h->off_v), h->base + h->off_weights, h->at<float>(h->off_status + 128), h->cfg.beta1, h->cfg.beta2, h->cfg.eps,
          h->cfg.weight_decay);
}

}  // extern "C"

// Runs `enqueue` (which puts one step's kernels on `st`) either directly or, when the stream allows capture (any
// stream but the legacy default one, not one the caller is capturing, no per-launch events asked for), as a CUDA graph
// captured on first use and replayed afterwards.
template <typename Enqueue>
static int run_step_graphed(bsr_handle* h, cudaStream_t st, const bsr_handle::StepGraph& key, Enqueue enqueue) {
  int rc;
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  bool can_graph = h->use_graph && st != nullptr && st != cudaStreamLegacy && !h->prof.on &&
                   cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone;
  auto direct = [&]() -> int {
    cudaGetLastError();
    int r = enqueue();
    return r != BSR_OK ? r : check_cuda(h, "training step");
  };
  if (!can_graph) return direct();
  for (auto& g : h->graphs) {
    if (g.images == key.images && g.labels == key.labels && g.tasks == key.tasks && g.loss == key.loss && g.kept == key.kept &&
        g.batch == key.batch && g.mode == key.mode && g.loop == key.loop) {
      g_kernel_launches += g.launches;
      g.last_use = ++h->graph_clock;
      if (cudaGraphLaunch(g.exec, st) != cudaSuccess) return set_err(h->err, BSR_ERR_CUDA, "graph launch failed: %s", cudaGetErrorString(cudaGetLastError()));
      return BSR_OK;
    }
  }
  long before = g_kernel_launches;
  if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) return direct();
  rc = enqueue();
  cudaGraph_t graph = nullptr;
  cudaError_t ce = cudaStreamEndCapture(st, &graph);
  if (rc != BSR_OK) {
    if (graph) cudaGraphDestroy(graph);
    return rc;
  }
  bsr_handle::StepGraph sg = key;
  sg.exec = nullptr; sg.launches = g_kernel_launches - before; sg.last_use = ++h->graph_clock;
  if (ce != cudaSuccess || graph == nullptr || cudaGraphInstantiate(&sg.exec, graph, 0) != cudaSuccess) {
    if (graph) cudaGraphDestroy(graph);
    return direct();                                     // nothing ran during the capture
  }
  cudaGraphDestroy(graph);
  ++h->graph_captures;
  if (h->graphs.size() >= bsr_handle::GRAPH_CACHE) {     // drop the least recently used graph
    size_t lru = 0;
    for (size_t i = 1; i < h->graphs.size(); ++i)
      if (h->graphs[i].last_use < h->graphs[lru].last_use) lru = i;
    cudaGraphExecDestroy(h->graphs[lru].exec);
    h->graphs.erase(h->graphs.begin() + lru);
  }
  h->graphs.push_back(sg);
  if (cudaGraphLaunch(sg.exec, st) != cudaSuccess) return set_err(h->err, BSR_ERR_CUDA, "graph launch failed: %s", cudaGetErrorString(cudaGetLastError()));
  return BSR_OK;
}

extern "C" {

int32_t bsr_train_step(bsr_handle* h, const void* images, const int32_t* labels, const int32_t* task_ids, int32_t batch,
                       void* stream, float* loss_out, int32_t* kept_out) {
  int rc = check_batch(h, images, batch);
  if (rc != BSR_OK) return rc;
  if (labels == nullptr || loss_out == nullptr) return set_err(h->err, BSR_ERR_INVALID_ARG, "labels_dev and loss_dev_out must not be null");
  if (h->cfg.dims.num_tasks > 1 && task_ids == nullptr) return set_err(h->err, BSR_ERR_INVALID_ARG, "task_ids_dev is required with several tasks");
  cudaStream_t st = (cudaStream_t)stream;
  // the step counter (AdamW's bias correction) advances only once the step has been enqueued
  const int64_t step_next = h->step + 1;
  double bc1 = 1.0 - std::pow((double)h->cfg.beta1, (double)step_next);
  double bc2 = 1.0 - std::pow((double)h->cfg.beta2, (double)step_next);
  set_scalars(st, h->at<float>(h->off_status + 128), h->lr, (float)bc1, (float)bc2);
  bsr_handle::StepGraph key;
  key.images = images; key.labels = labels; key.tasks = task_ids; key.loss = loss_out; key.kept = kept_out; key.batch = batch;
  key.mode = h->use_tc; key.loop = 0; key.exec = nullptr; key.launches = 0; key.last_use = 0;
  rc = run_step_graphed(h, st, key, [&]() { return enqueue_train_step(h, images, labels, task_ids, batch, stream, loss_out, kept_out); });
  if (rc == BSR_OK) h->step = step_next;
  return rc;
}

int32_t bsr_forward_backward(bsr_handle* h, const void* images, const int32_t* labels, const int32_t* task_ids, int32_t batch,
                             void* stream, float* loss_out, int32_t* kept_out) {
  int rc = check_batch(h, images, batch);
  if (rc != BSR_OK) return rc;
  if (labels == nullptr || loss_out == nullptr) return set_err(h->err, BSR_ERR_INVALID_ARG, "labels_dev and loss_dev_out must not be null");
  if (h->cfg.dims.num_tasks > 1 && task_ids == nullptr) return set_err(h->err, BSR_ERR_INVALID_ARG, "task_ids_dev is required with several tasks");
  bsr_handle::StepGraph key;
  key.images = images; key.labels = labels; key.tasks = task_ids; key.loss = loss_out; key.kept = kept_out; key.batch = batch;
  key.mode = h->use_tc; key.loop = 2; key.exec = nullptr; key.launches = 0; key.last_use = 0;
  return run_step_graphed(h, (cudaStream_t)stream, key, [&]() {
    return enqueue_train_step(h, images, labels, task_ids, batch, stream, loss_out, kept_out, nullptr, false);
  });
}

int32_t bsr_grad_buffer(bsr_handle* h, float** grads_dev_out, size_t* count_out) {
  if (h == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "handle is null");
  if (grads_dev_out == nullptr || count_out == nullptr) return set_err(h->err, BSR_ERR_INVALID_ARG, "null argument");
  *grads_dev_out = h->at<float>(h->off_grad);
  *count_out = h->n_flat;
  return BSR_OK;
}

int32_t bsr_optimizer_step(bsr_handle* h, void* stream) {
  if (h == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "handle is null");
  cudaStream_t st = (cudaStream_t)stream;
  const int64_t step_next = h->step + 1;
  double bc1 = 1.0 - std::pow((double)h->cfg.beta1, (double)step_next);
  double bc2 = 1.0 - std::pow((double)h->cfg.beta2, (double)step_next);
  set_scalars(st, h->at<float>(h->off_status + 128), h->lr, (float)bc1, (float)bc2);
  Ctx c = make_ctx(h, stream);
  enqueue_optimizer(h, c);
  int rc = check_cuda(h, "bsr_optimizer_step");
  if (rc == BSR_OK) h->step = step_next;
  return rc;
}

int32_t bsr_train_steps(bsr_handle* h, const void* images, const int32_t* labels, const int32_t* task_ids, int32_t batch,
                        int32_t n_steps, const bsr_lr_schedule* sched, void* stream, float* loss_out, int32_t* kept_out) {
  int rc = check_batch(h, images, batch);
  if (rc != BSR_OK) return rc;
  if (labels == nullptr || loss_out == nullptr || sched == nullptr) return set_err(h->err, BSR_ERR_INVALID_ARG, "labels_dev, loss_dev_out and schedule must not be null");
  if (h->cfg.dims.num_tasks > 1 && task_ids == nullptr) return set_err(h->err, BSR_ERR_INVALID_ARG, "task_ids_dev is required with several tasks");
  if (n_steps < 1) return set_err(h->err, BSR_ERR_INVALID_ARG, "n_steps must be positive");
  if (sched->total_steps < 1 || !(sched->lr_max >= sched->lr_min) || !(sched->lr_min >= 0.f))
    return set_err(h->err, BSR_ERR_INVALID_ARG, "schedule needs total_steps >= 1 and lr_max >= lr_min >= 0");
  const bsr_dims& d = h->cfg.dims;
  cudaStream_t st = (cudaStream_t)stream;
  LoopState* ls = h->at<LoopState>(h->off_loop);
  long long stride = (long long)batch * d.in_chans * d.image_size * d.image_size;
  loop_init(st, ls, h->step, sched->total_steps, stride, sched->lr_max, sched->lr_min, h->cfg.beta1, h->cfg.beta2, n_steps);
  int* lab_stage = h->at<int>(h->off_lab_stage);
  int* task_stage = task_ids != nullptr ? h->at<int>(h->off_task_stage) : nullptr;
  float* scalars = h->at<float>(h->off_status + 128);
  bsr_handle::StepGraph key;
  key.images = images; key.labels = labels; key.tasks = task_ids; key.loss = loss_out; key.kept = kept_out; key.batch = batch;
  key.mode = h->use_tc; key.loop = 1; key.exec = nullptr; key.launches = 0; key.last_use = 0;
  for (int i = 0; i < n_steps; ++i) {
    rc = run_step_graphed(h, st, key, [&]() {
      loop_begin(st, ls, scalars, labels, task_ids, lab_stage, task_stage, batch);
      int r = enqueue_train_step(h, images, lab_stage, task_stage, batch, stream, nullptr, kept_out, &ls->image_offset);
      loop_end(st, ls, h->at<float>(h->off_loss), loss_out);
      return r;
    });
    if (rc != BSR_OK) return rc;
    h->step += 1;
  }
  // the schedule's last learning rate stays in force for later single steps
  double frac = (double)(h->step - 1 < sched->total_steps ? h->step - 1 : sched->total_steps) / (double)sched->total_steps;
  h->lr = (float)((double)sched->lr_min + 0.5 * ((double)sched->lr_max - (double)sched->lr_min) * (1.0 + std::cos(3.14159265358979323846 * frac)));
  return BSR_OK;
}

int32_t bsr_train_step_host(bsr_handle* h, const void* images_host, const int32_t* labels_host, const int32_t* task_ids_host,
                            int32_t batch, void* stream, float* loss_host_out, int32_t* kept_host_out) {
  int rc = check_batch(h, images_host, batch);
  if (rc != BSR_OK) return rc;
  if (labels_host == nullptr || loss_host_out == nullptr) return set_err(h->err, BSR_ERR_INVALID_ARG, "labels_host and loss_host_out must not be null");
  if (h->cfg.dims.num_tasks > 1 && task_ids_host == nullptr) return set_err(h->err, BSR_ERR_INVALID_ARG, "task_ids_host is required with several tasks");
  const bsr_dims& d = h->cfg.dims;
  cudaStream_t st = (cudaStream_t)stream;
  if (h->copy_stream == nullptr) {                       // host objects, created on first use
    bool ok = cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i)
      ok = cudaEventCreateWithFlags(&h->ev_copied[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&h->ev_done[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) return set_err(h->err, BSR_ERR_CUDA, "could not create the copy stream: %s", cudaGetErrorString(cudaGetLastError()));
  }
  int slot = h->host_slot;
  h->host_slot ^= 1;
  // The inputs travel on the library's copy stream into one of two staging slots, so that the copy for this step
  // overlaps the previous step's kernels; the slot's previous user (two calls back) must have finished with it.
  if (h->slot_used[slot]) cudaStreamWaitEvent(h->copy_stream, h->ev_done[slot], 0);
  size_t img_bytes = (size_t)batch * d.in_chans * d.image_size * d.image_size * dtype_size(d.dtype);
  void* img_dev = h->base + h->off_host_img[slot];
  int32_t* lab_dev = h->at<int32_t>(h->off_host_lab[slot]);
  int32_t* task_dev = task_ids_host != nullptr ? h->at<int32_t>(h->off_host_task[slot]) : nullptr;
  float* loss_dev = h->at<float>(h->off_host_loss[slot]);
  cudaMemcpyAsync(img_dev, images_host, img_bytes, cudaMemcpyHostToDevice, h->copy_stream);
  cudaMemcpyAsync(lab_dev, labels_host, (size_t)batch * 4, cudaMemcpyHostToDevice, h->copy_stream);
  if (task_dev != nullptr) cudaMemcpyAsync(task_dev, task_ids_host, (size_t)batch * 4, cudaMemcpyHostToDevice, h->copy_stream);
  cudaEventRecord(h->ev_copied[slot], h->copy_stream);
  cudaStreamWaitEvent(st, h->ev_copied[slot], 0);
  rc = bsr_train_step(h, img_dev, lab_dev, task_dev, batch, stream, loss_dev, nullptr);
  if (rc != BSR_OK) return rc;
  cudaMemcpyAsync(loss_host_out, loss_dev, 4, cudaMemcpyDeviceToHost, st);
  if (kept_host_out != nullptr && kept_total(h, batch) > 0)
    cudaMemcpyAsync(kept_host_out, h->base + h->off_kept_all, kept_total(h, batch) * 4, cudaMemcpyDeviceToHost, st);
  cudaEventRecord(h->ev_done[slot], st);
  h->slot_used[slot] = true;
  return check_cuda(h, "bsr_train_step_host");
}

int32_t bsr_eval_forward(bsr_handle* h, const void* images, const int32_t* task_ids, int32_t batch, void* stream,
                         float* logits_out, int32_t* kept_out) {
  int rc = check_batch(h, images, batch);
  if (rc != BSR_OK) return rc;
  if (logits_out == nullptr) return set_err(h->err, BSR_ERR_INVALID_ARG, "logits_dev_out is null");
  if (h->cfg.dims.num_tasks > 1 && task_ids == nullptr) return set_err(h->err, BSR_ERR_INVALID_ARG, "task_ids_dev is required with several tasks");
  const bsr_dims& d = h->cfg.dims;
  Ctx c = make_ctx(h, stream);
  size_t x_last = 0;
  rc = forward_all(h, c, images, batch, false, &x_last, task_ids);
  if (rc != BSR_OK) return rc;
  int Tl = cls_tail(h, d.depth - 1) ? 1 : h->sched.tf[d.depth - 1];   // rows per image in the last block's output
  HeadDesc hd = head_desc(h);
  float* xn = h->at<float>(h->off_xn);
  layernorm_fwd(c, h->at<float>(x_last), (long)Tl * d.dim, (const float*)h->w("norm.weight"), (const float*)h->w("norm.bias"), xn, 1,
                nullptr, nullptr, batch, d.dim, d.ln_eps);
  head_fwd(c, hd, xn, task_ids, h->at<float>(h->off_logits), batch);
  cudaMemcpyAsync(logits_out, h->at<float>(h->off_logits), (size_t)batch * hd.cmax * 4, cudaMemcpyDeviceToDevice, c.stream);
  if (kept_out != nullptr && kept_total(h, batch) > 0)
    cudaMemcpyAsync(kept_out, h->base + h->off_kept_all, kept_total(h, batch) * 4, cudaMemcpyDeviceToDevice, c.stream);
  return check_cuda(h, "bsr_eval_forward");
}

int32_t bsr_get_footprint(const bsr_handle* h, bsr_footprint* out) {
  if (h == nullptr || out == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "null argument");
  const bsr_dims& d = h->cfg.dims;
  memset(out, 0, sizeof(*out));
  out->workspace_bytes = h->bytes;
  out->weight_bytes = h->weights_bytes;
  out->master_bytes = h->n_flat * 4;
  out->optimizer_bytes = h->n_flat * 8;
  out->grad_bytes = h->n_flat * 4;
  out->saved_activation_bytes = h->arena_bytes;
  out->scratch_bytes = h->scratch_bytes;
  uint64_t paper = 0, params = 0;
  for (int l = h->t0; l < d.depth; ++l) {
    // Table 1 accounting in fp32: Q,K,V + softmax input + GELU input, plus the inputs of the six linear layers
    uint64_t ta = h->sched.ta[l], tf = h->sched.tf[l];
    uint64_t el = 3 * ta * d.dim + (uint64_t)d.heads * ta * ta + tf * d.mlp_hidden;
    if ((h->cfg.trainable_mask >> l) & 1u) el += 3 * ta * d.dim + 2 * tf * d.dim + tf * d.mlp_hidden;   // inputs of the linear layers
    paper += el * 4 * (uint64_t)h->cfg.max_batch;
  }
  for (auto& t : h->tensors)
    if (t.trainable) params += t.numel;
  out->paper_activation_bytes = paper;
  out->trainable_params = params;
  for (int l = 0; l < d.depth && l < BSR_MAX_DEPTH; ++l) out->block_saved_bytes[l] = h->block_saved_bytes[l];
  return BSR_OK;
}

int32_t bsr_sync_status(bsr_handle* h, void* stream) {
  if (h == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "handle is null");
  int st = 0;
  if (!h->guards.empty())
    guards_check((cudaStream_t)stream, h->base, h->at<unsigned long long>(h->off_guard_table), (int)h->guards.size(), (int)(GUARD_BYTES / 4),
                 GUARD_WORD, h->at<int>(h->off_status));
  cudaError_t e = cudaMemcpyAsync(&st, h->base + h->off_status, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(h->base + h->off_status, 0, 4, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) return set_err(h->err, BSR_ERR_CUDA, "bsr_sync_status: %s", cudaGetErrorString(e));
  if (st & STATUS_TIMEOUT) return set_err(h->err, BSR_ERR_DEVICE_TIMEOUT, "a bounded device-side wait expired");
  if (st & STATUS_GUARD) return set_err(h->err, BSR_ERR_MEMORY_GUARD, "a guard word between two workspace slices was overwritten");
  if (st & STATUS_CHECK) return set_err(h->err, BSR_ERR_DEVICE_CHECK, "a device-side index check failed (checked build)");
  if (st & STATUS_NONFINITE) return set_err(h->err, BSR_ERR_NONFINITE, "the loss was not finite");
  return BSR_OK;
}

int32_t bsr_selftest_wait_expiry(bsr_handle* h, uint64_t limit_ns, void* stream) {
  if (h == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "handle is null");
  if (limit_ns < 1000 || limit_ns > 100000000ull) return set_err(h->err, BSR_ERR_INVALID_ARG, "limit_ns must lie in [1e3, 1e8]");
  if (h->cfg.dims.dtype != BSR_DTYPE_BF16) return set_err(h->err, BSR_ERR_UNSUPPORTED, "only bf16 handles run kernels with bounded waits");
  Ctx c = make_ctx(h, stream);
  wait_expiry_selftest(c, limit_ns);
  return check_cuda(h, "bsr_selftest_wait_expiry");
}

int32_t bsr_set_gemm_mode(bsr_handle* h, int32_t mode) {
  if (h == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "handle is null");
  if (mode < 0 || mode > 2) return set_err(h->err, BSR_ERR_INVALID_ARG, "mode must be 0, 1 or 2");
  h->use_tc = mode;
  return BSR_OK;
}

int32_t bsr_set_graph_mode(bsr_handle* h, int32_t on) {
  if (h == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "handle is null");
  h->use_graph = on != 0;
  return BSR_OK;
}

int32_t bsr_profile_enable(bsr_handle* h, int32_t time_gemms) {
  if (h == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "handle is null");
  h->prof.on = time_gemms != 0;
  h->prof.used = 0;
  h->prof.flops = 0.0;
  h->prof.launch_flops.clear();
  h->launches_at_enable = g_kernel_launches;
  return BSR_OK;
}

int32_t bsr_profile_read(bsr_handle* h, void* stream, bsr_profile* out) {
  if (h == nullptr || out == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "null argument");
  cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) return set_err(h->err, BSR_ERR_CUDA, "bsr_profile_read: %s", cudaGetErrorString(e));
  double ms = 0.0;
  for (size_t i = 0; i + 1 < h->prof.used; i += 2) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, h->prof.events[i], h->prof.events[i + 1]) == cudaSuccess) ms += t;
  }
  out->kernel_launches = (uint64_t)(g_kernel_launches - h->launches_at_enable);
  out->gemm_launches = h->prof.used / 2;
  out->gemm_flops = h->prof.flops;
  out->gemm_ms = ms;
  out->graph_captures = h->graph_captures;
  return BSR_OK;
}

int32_t bsr_profile_launches(bsr_handle* h, void* stream, int32_t capacity, double* flops_out, float* ms_out, int32_t* count_out) {
  if (h == nullptr || flops_out == nullptr || ms_out == nullptr || count_out == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "null argument");
  cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) return set_err(h->err, BSR_ERR_CUDA, "bsr_profile_launches: %s", cudaGetErrorString(e));
  int n = (int)(h->prof.used / 2);
  *count_out = n;
  for (int i = 0; i < n && i < capacity; ++i) {
    float t = 0.f;
    cudaEventElapsedTime(&t, h->prof.events[2 * i], h->prof.events[2 * i + 1]);
    ms_out[i] = t;
    flops_out[i] = h->prof.launch_flops[i];
  }
  return BSR_OK;
}

// ---- stand-alone kernels ------------------------------------------------------------------------

static Ctx bare_ctx(int dtype, void* stream) {
  Ctx c;
  c.stream = (cudaStream_t)stream;
  c.dtype = dtype;
  c.status = nullptr;
  c.sm_count = 0;
  c.use_tc = 0;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess) c.sm_count = sms;
  return c;
}

int32_t bsr_token_select(const float* p, int32_t batch, int32_t heads, int32_t m, int32_t k, float* scores, int32_t* kept,
                         int32_t* dropped, void* stream) {
  if (p == nullptr || scores == nullptr || kept == nullptr || (dropped == nullptr && k < m)) return set_err(g_error, BSR_ERR_INVALID_ARG, "null argument");
  if (batch < 1 || heads < 1 || m < 1 || m > 4096 || k < 1 || k > m) return set_err(g_error, BSR_ERR_INVALID_ARG, "need batch, heads >= 1 and 1 <= k <= m <= 4096");
  token_select((cudaStream_t)stream, p, batch, heads, m, k, scores, kept, dropped);
  return check_cuda(nullptr, "bsr_token_select");
}

int32_t bsr_gather_fuse(const void* x, int32_t dtype, int32_t batch, int32_t m, int32_t dim, int32_t k, const int32_t* kept,
                        const int32_t* dropped, const float* scores, int32_t fuse_mode, void* out, void* stream) {
  if (x == nullptr || kept == nullptr || out == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "null argument");
  if (dtype != BSR_DTYPE_FP32 && dtype != BSR_DTYPE_BF16) return set_err(g_error, BSR_ERR_INVALID_ARG, "bad dtype");
  if (batch < 1 || m < 1 || k < 1 || k > m || dim < 1 || (dim * dtype_size(dtype)) % 16 != 0) return set_err(g_error, BSR_ERR_INVALID_ARG, "bad shape: rows must be a multiple of 16 bytes, 1 <= k <= m");
  bool fuse = (fuse_mode == BSR_FUSE_WEIGHTED_SUM || fuse_mode == BSR_FUSE_WEIGHTED_MEAN) && k < m;
  if (fuse && (dropped == nullptr || scores == nullptr)) return set_err(g_error, BSR_ERR_INVALID_ARG, "fusion needs dropped_dev and scores_dev");
  Ctx c = bare_ctx(dtype, stream);
  gather_fuse(c, x, batch, m, dim, k, kept, dropped, scores, fuse_mode, out);
  return check_cuda(nullptr, "bsr_gather_fuse");
}

int32_t bsr_linear_forward(const void* x, const void* w, const float* bias, const void* residual, void* y, int32_t m, int32_t n,
                           int32_t k, int32_t dtype, int32_t act_gelu, int32_t use_tensor_cores, void* stream) {
  if (x == nullptr || w == nullptr || y == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "null argument");
  if (dtype != BSR_DTYPE_FP32 && dtype != BSR_DTYPE_BF16) return set_err(g_error, BSR_ERR_INVALID_ARG, "bad dtype");
  if (m < 1 || n < 1 || k < 1) return set_err(g_error, BSR_ERR_INVALID_ARG, "bad shape");
  Ctx c = bare_ctx(dtype, stream);
  GemmEpilogue e;
  e.bias = bias;
  e.residual = residual;
  e.act = act_gelu ? 1 : 0;
  if (use_tensor_cores) {
    if (dtype != BSR_DTYPE_BF16 || !gemm_tc_supported(m, n, k)) return set_err(g_error, BSR_ERR_UNSUPPORTED, "the tcgen05 kernel needs bf16 and k, n multiples of 8");
    int rc = use_tensor_cores >= 2 ? gemm_tc2_strided(c, x, k, 1, w, k, 1, y, 0, m, n, k, e, nullptr, 0) : gemm_tc(c, x, w, y, 0, m, n, k, e);
    if (rc != 0) return set_err(g_error, BSR_ERR_CUDA, "tcgen05 GEMM set-up failed (%d)", rc);
  } else {
    gemm(c, x, k, 1, w, k, 1, y, 0, m, n, k, e);
  }
  return check_cuda(nullptr, "bsr_linear_forward");
}

int32_t bsr_linear_forward_e4m3(const void* x, const void* w, const float* bias, void* y, int32_t m, int32_t n, int32_t k,
                                int32_t act_gelu, void* scratch, size_t scratch_bytes, void* stream) {
  if (x == nullptr || w == nullptr || y == nullptr || scratch == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "null argument");
  if (m < 1 || n < 8 || k < 16 || (k % 16) || (n % 8)) return set_err(g_error, BSR_ERR_INVALID_ARG, "need k a multiple of 16 and n a multiple of 8");
  auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
  size_t o_xq = 0, o_wq = o_xq + up((size_t)m * k), o_xs = o_wq + up((size_t)n * k), o_ws = o_xs + up((size_t)m * 4), need = o_ws + up((size_t)n * 4);
  if (((uintptr_t)scratch & 255) != 0 || scratch_bytes < need) return set_err(g_error, BSR_ERR_WORKSPACE_TOO_SMALL, "scratch of %zu bytes given, %zu needed (256-byte aligned)", scratch_bytes, need);
  Ctx c = bare_ctx(BSR_DTYPE_BF16, stream);
  c.use_tc = 1;
  char* s0 = (char*)scratch;
  quantize_rows_e4m3(c, x, m, k, s0 + o_xq, (float*)(s0 + o_xs));
  quantize_rows_e4m3(c, w, n, k, s0 + o_wq, (float*)(s0 + o_ws));
  GemmEpilogue e;
  e.bias = bias;
  e.act = act_gelu ? 1 : 0;
  if (gemm_tc_e4m3(c, s0 + o_xq, (const float*)(s0 + o_xs), s0 + o_wq, (const float*)(s0 + o_ws), y, m, n, k, e) != 0)
    return set_err(g_error, BSR_ERR_CUDA, "8-bit GEMM set-up failed");
  return check_cuda(nullptr, "bsr_linear_forward_e4m3");
}

int32_t bsr_linear_backward(const void* x, const void* w, const void* dy, void* dx, float* dw, int32_t m, int32_t n, int32_t k,
                            int32_t dtype, int32_t use_tensor_cores, float* workspace, size_t workspace_floats, void* stream) {
  if (x == nullptr || w == nullptr || dy == nullptr || dx == nullptr || dw == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "null argument");
  if (dtype != BSR_DTYPE_FP32 && dtype != BSR_DTYPE_BF16) return set_err(g_error, BSR_ERR_INVALID_ARG, "bad dtype");
  if (m < 1 || n < 1 || k < 1) return set_err(g_error, BSR_ERR_INVALID_ARG, "bad shape");
  Ctx c = bare_ctx(dtype, stream);
  GemmEpilogue none;
  if (use_tensor_cores) {
    if (dtype != BSR_DTYPE_BF16 || (m % 8) || (n % 8) || (k % 8)) return set_err(g_error, BSR_ERR_UNSUPPORTED, "the tcgen05 kernels need bf16 and m, n, k multiples of 8");
    int rc;
    if (use_tensor_cores >= 2) {
      rc = gemm_tc2_strided(c, dy, n, 1, w, 1, k, dx, 0, m, k, n, none, nullptr, 0);
      if (rc == 0) rc = gemm_tc2_strided(c, dy, 1, n, x, 1, k, dw, 1, n, k, m, none, workspace, workspace_floats);
    } else {
      rc = gemm_tc_strided(c, dy, n, 1, w, 1, k, dx, 0, m, k, n, none, nullptr, 0);                       // dX = dY W
      if (rc == 0) rc = gemm_tc_strided(c, dy, 1, n, x, 1, k, dw, 1, n, k, m, none, workspace, workspace_floats);   // dW = dY^T X
    }
    if (rc != 0) return set_err(g_error, BSR_ERR_CUDA, "tcgen05 GEMM set-up failed (%d)", rc);
  } else {
    gemm(c, dy, n, 1, w, 1, k, dx, 0, m, k, n, none);
    gemm(c, dy, 1, n, x, 1, k, dw, 1, n, k, m, none);
  }
  return check_cuda(nullptr, "bsr_linear_backward");
}

int32_t bsr_attention_forward(const void* qkv, int32_t dtype, int32_t batch, int32_t t, int32_t heads, int32_t d, void* out,
                              float* cls_prob, float* lse, int32_t use_tensor_cores, void* stream) {
  if (qkv == nullptr || out == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "null argument");
  if (dtype != BSR_DTYPE_FP32 && dtype != BSR_DTYPE_BF16) return set_err(g_error, BSR_ERR_INVALID_ARG, "bad dtype");
  if (batch < 1 || t < 1 || heads < 1 || d < 8 || d > 64 || d % 8 != 0) return set_err(g_error, BSR_ERR_INVALID_ARG, "bad shape: head dimension must be a multiple of 8, at most 64");
  Ctx c = bare_ctx(dtype, stream);
  if (use_tensor_cores) {
    if (attention_fwd_tc(c, qkv, out, lse, cls_prob, batch, t, heads, d) != 0)
      return set_err(g_error, BSR_ERR_UNSUPPORTED, "the tcgen05 attention kernels need bf16 and head dimension 64");
    return check_cuda(nullptr, "bsr_attention_forward");
  }
  if (attention_fwd(c, qkv, out, lse, cls_prob, batch, t, heads, d) != 0)
    return set_err(g_error, BSR_ERR_UNSUPPORTED, "%d tokens do not fit the attention kernel's shared memory", t);
  return check_cuda(nullptr, "bsr_attention_forward");
}

int32_t bsr_attention_backward(const void* qkv, const void* dout, const float* lse, const float* score_grad, int32_t dtype,
                               int32_t batch, int32_t t, int32_t heads, int32_t d, void* dqkv, float* delta_scratch,
                               int32_t use_tensor_cores, void* stream) {
  if (qkv == nullptr || dout == nullptr || lse == nullptr || dqkv == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "null argument");
  if (dtype != BSR_DTYPE_FP32 && dtype != BSR_DTYPE_BF16) return set_err(g_error, BSR_ERR_INVALID_ARG, "bad dtype");
  if (batch < 1 || t < 1 || heads < 1 || d < 8 || d > 64 || d % 8 != 0) return set_err(g_error, BSR_ERR_INVALID_ARG, "bad shape: head dimension must be a multiple of 8, at most 64");
  Ctx c = bare_ctx(dtype, stream);
  if (use_tensor_cores) {
    if (attention_bwd_tc(c, qkv, dout, lse, score_grad, dqkv, batch, t, heads, d) != 0)
      return set_err(g_error, BSR_ERR_UNSUPPORTED, "the tcgen05 attention backward needs bf16, head dimension 64 and at most 256 tokens");
    return check_cuda(nullptr, "bsr_attention_backward");
  }
  if (delta_scratch == nullptr) return set_err(g_error, BSR_ERR_INVALID_ARG, "delta_scratch_dev is required without tensor cores");
  c.use_tc = 0;
  if (attention_bwd(c, qkv, nullptr, dout, lse, delta_scratch, score_grad, dqkv, batch, t, heads, d) != 0)
    return set_err(g_error, BSR_ERR_UNSUPPORTED, "%d tokens do not fit the attention kernel's shared memory", t);
  return check_cuda(nullptr, "bsr_attention_backward");
}

}  // extern "C"
