// Host-side description of the network behind an lp_net_desc: blocks, module split, boundary
// shapes, AuxNet shapes and the flat parameter layouts.  Pure host code (no CUDA).
#pragma once
#include <stdio.h>
#include <string.h>

#include <string>
#include <vector>

#include "../../include/lp.h"

namespace lp {

struct BlockDef {
  int cin, cout, stride, hin, win, hout, wout;
  bool proj;
  int mid;   // inner width of a bottleneck block (C_out / 4)
};
struct AuxConvDef {
  int cin, cout, stride, hin, win, hout, wout;
};
struct Shape4 {
  int n, h, w, c;
  long long elems() const { return (long long)n * h * w * c; }
};

inline int conv_out(int h, int r, int stride, int pad) { return (h + 2 * pad - r) / stride + 1; }

struct NetDef {
  lp_net_desc d;
  int K = 0;
  int stem_R = 3, stem_stride = 1, stem_pad = 1;
  bool stem_pool = false;
  int stem_h = 0, stem_w = 0;      // stem conv output
  int body_h = 0, body_w = 0;      // input of block 0 (after the optional max-pool)
  std::vector<BlockDef> blocks;
  std::vector<int> mod_begin, mod_end;
  std::vector<Shape4> boundary;     // x_k, k = 0..K-1
  std::vector<std::vector<AuxConvDef>> aux;

  int build(const lp_net_desc* desc) {
    if (!desc) return LP_ERR_NULL;
    if (desc->struct_size != sizeof(lp_net_desc)) return LP_ERR_BAD_DESC;
    d = *desc;
    if (d.dtype != LP_F32 && d.dtype != LP_BF16) return LP_ERR_BAD_DESC;
    if (d.N < 1 || d.H < 1 || d.W < 1 || d.C_in < 1 || d.num_classes < 2) return LP_ERR_BAD_DESC;
    if (d.stem_kind != LP_STEM_CONV3X3 && d.stem_kind != LP_STEM_CONV7X7S2_MAXPOOL) return LP_ERR_BAD_DESC;
    if (d.block_kind != LP_POSTBN && d.block_kind != LP_PREACT && d.block_kind != LP_BOTTLENECK) return LP_ERR_BAD_DESC;
    if (d.post_add_relu != 0) return LP_ERR_UNSUPPORTED;
    if (d.num_stages < 1 || d.num_stages > LP_MAX_STAGES) return LP_ERR_BAD_DESC;
    if (d.K < 1 || d.K > LP_MAX_MODULES) return LP_ERR_BAD_DESC;
    if (d.aux_convs_per_boundary < 1 || d.aux_convs_per_boundary > 2 || d.aux_width_div < 1) return LP_ERR_BAD_DESC;
    if (!(d.bn_eps > 0.f)) return LP_ERR_BAD_DESC;
    if (d.aux_recursive != 0 && d.aux_recursive != 1) return LP_ERR_BAD_DESC;
    if (d.conv_impl < 0 || (d.conv_impl & 15) > LP_CONV_IMPL_TENSOR || d.conv_impl > 8191) return LP_ERR_BAD_DESC;
    const int vec = d.dtype == LP_F32 ? 4 : 8;
    if (d.stem_channels < vec || d.stem_channels % vec) return LP_ERR_BAD_DESC;
    if (d.stem_kind == LP_STEM_CONV7X7S2_MAXPOOL && d.block_kind == LP_PREACT) return LP_ERR_UNSUPPORTED;
    K = d.K;
    int h = d.H, w = d.W;
    if (d.stem_kind == LP_STEM_CONV7X7S2_MAXPOOL) {
      stem_R = 7; stem_stride = 2; stem_pad = 3; stem_pool = true;
      h = conv_out(h, 7, 2, 3); w = conv_out(w, 7, 2, 3);
      stem_h = h; stem_w = w;
      h = conv_out(h, 3, 2, 1); w = conv_out(w, 3, 2, 1);
    } else {
      stem_h = h; stem_w = w;
    }
    if (h < 1 || w < 1) return LP_ERR_BAD_DESC;
    body_h = h; body_w = w;
    int c = d.stem_channels;
    blocks.clear();
    for (int s = 0; s < d.num_stages; ++s) {
      const int ch = d.stage_channels[s], nb = d.stage_blocks[s], st = d.stage_stride[s];
      if (ch < vec || ch % vec || nb < 1 || (st != 1 && st != 2)) return LP_ERR_BAD_DESC;
      for (int b = 0; b < nb; ++b) {
        BlockDef bd;
        bd.cin = c; bd.cout = ch; bd.stride = b == 0 ? st : 1;
        bd.hin = h; bd.win = w;
        bd.proj = bd.stride != 1 || c != ch;
        bd.mid = ch / 4;
        if (d.block_kind == LP_BOTTLENECK && (ch % 4 || bd.mid < vec || bd.mid % vec)) return LP_ERR_BAD_DESC;
        h = conv_out(h, 3, bd.stride, 1); w = conv_out(w, 3, bd.stride, 1);
        if (h < 1 || w < 1) return LP_ERR_BAD_DESC;
        bd.hout = h; bd.wout = w;
        blocks.push_back(bd);
        c = ch;
      }
    }
    mod_begin.clear(); mod_end.clear();
    int prev = 0;
    for (int k = 0; k < K; ++k) {
      const int e = d.module_block_end[k];
      if (e <= prev || e > (int)blocks.size()) return LP_ERR_BAD_DESC;
      mod_begin.push_back(prev); mod_end.push_back(e);
      prev = e;
    }
    if (prev != (int)blocks.size()) return LP_ERR_BAD_DESC;
    boundary.clear();
    boundary.push_back(Shape4{d.N, d.H, d.W, d.C_in});
    for (int k = 1; k < K; ++k) {
      const BlockDef& b = blocks[mod_begin[k]];
      boundary.push_back(Shape4{d.N, b.hin, b.win, b.cin});
    }
    aux.clear();
    for (int k = 0; k + 1 < K; ++k) {
      const Shape4 a = boundary[k], o = boundary[k + 1];
      if (o.h < 1 || a.h % o.h || a.w % o.w || a.h / o.h != a.w / o.w) return LP_ERR_BAD_DESC;
      const int total = a.h / o.h;
      std::vector<AuxConvDef> cv;
      if (d.aux_convs_per_boundary == 1) {
        if (total != 1 && total != 2) return LP_ERR_BAD_DESC;
        cv.push_back(AuxConvDef{a.c, o.c, total, a.h, a.w, o.h, o.w});
      } else {
        if (total != 1 && total != 2 && total != 4) return LP_ERR_BAD_DESC;
        int hid = o.c / d.aux_width_div;
        if (hid < vec || hid % vec) return LP_ERR_BAD_DESC;
        const int s1 = total >= 2 ? 2 : 1, s2 = total == 4 ? 2 : 1;
        const int mh = conv_out(a.h, 3, s1, 1), mw = conv_out(a.w, 3, s1, 1);
        cv.push_back(AuxConvDef{a.c, hid, s1, a.h, a.w, mh, mw});
        cv.push_back(AuxConvDef{hid, o.c, s2, mh, mw, conv_out(mh, 3, s2, 1), conv_out(mw, 3, s2, 1)});
        if (cv[1].hout != o.h || cv[1].wout != o.w) return LP_ERR_BAD_DESC;
      }
      aux.push_back(cv);
    }
    return LP_OK;
  }

  static void push(std::vector<lp_param_entry>& L, uint64_t& off, const std::string& name, int kind, int s0,
                   int s1 = 0, int s2 = 0, int s3 = 0) {
    lp_param_entry e;
    memset(&e, 0, sizeof(e));
    snprintf(e.name, sizeof(e.name), "%s", name.c_str());
    e.kind = kind;
    e.shape[0] = s0; e.shape[1] = s1; e.shape[2] = s2; e.shape[3] = s3;
    e.offset = off;
    uint64_t n = (uint64_t)s0;
    if (s1) n *= s1;
    if (s2) n *= s2;
    if (s3) n *= s3;
    off += n;
    L.push_back(e);
  }

  // Flat parameter layout (blob order) of module `which` or AuxNet LP_AUX(k).
  // AuxNet plans: the K-1 networks of the chain, or (recursive form) the units of the K-1 stacks,
  // stack k = 1..K-1 holding units j = 0..k-1 at index k(k-1)/2 + j; a unit has AuxNet_j's shape.
  int n_aux_plans() const { return K < 2 ? 0 : (d.aux_recursive ? K * (K - 1) / 2 : K - 1); }
  static int reaux_index(int k, int j) { return k * (k - 1) / 2 + j; }
  int aux_unit(int idx) const {
    if (!d.aux_recursive) return idx;
    int k = 1;
    while (reaux_index(k + 1, 0) <= idx) ++k;
    return idx - reaux_index(k, 0);
  }

  int layout(int which, std::vector<lp_param_entry>& L, uint64_t* total) const {
    L.clear();
    uint64_t off = 0;
    if (which >= LP_AUX(0)) {
      const int idx = which - LP_AUX(0);
      if (idx < 0 || idx >= n_aux_plans()) return LP_ERR_BAD_INDEX;
      const int k = aux_unit(idx);
      for (size_t i = 0; i < aux[k].size(); ++i) {
        const std::string id = std::to_string(i + 1);
        push(L, off, "conv" + id + ".w", LP_KIND_CONV_W, aux[k][i].cout, 3, 3, aux[k][i].cin);
        push(L, off, "bn" + id + ".g", LP_KIND_BN_GAMMA, aux[k][i].cout);
        push(L, off, "bn" + id + ".b", LP_KIND_BN_BETA, aux[k][i].cout);
      }
      if (total) *total = off;
      return LP_OK;
    }
    const int k = which;
    if (k < 0 || k >= K) return LP_ERR_BAD_INDEX;
    const bool post = d.block_kind != LP_PREACT;
    const bool bott = d.block_kind == LP_BOTTLENECK;
    if (k == 0) {
      push(L, off, "stem.conv.w", LP_KIND_CONV_W, d.stem_channels, stem_R, stem_R, d.C_in);
      if (post) {
        push(L, off, "stem.bn.g", LP_KIND_BN_GAMMA, d.stem_channels);
        push(L, off, "stem.bn.b", LP_KIND_BN_BETA, d.stem_channels);
      }
    }
    for (int bi = mod_begin[k]; bi < mod_end[k]; ++bi) {
      const BlockDef& b = blocks[bi];
      const std::string p = "block" + std::to_string(bi) + ".";
      if (bott) {
        push(L, off, p + "conv1.w", LP_KIND_CONV_W, b.mid, 1, 1, b.cin);
        push(L, off, p + "bn1.g", LP_KIND_BN_GAMMA, b.mid);
        push(L, off, p + "bn1.b", LP_KIND_BN_BETA, b.mid);
        push(L, off, p + "conv2.w", LP_KIND_CONV_W, b.mid, 3, 3, b.mid);
        push(L, off, p + "bn2.g", LP_KIND_BN_GAMMA, b.mid);
        push(L, off, p + "bn2.b", LP_KIND_BN_BETA, b.mid);
        push(L, off, p + "conv3.w", LP_KIND_CONV_W, b.cout, 1, 1, b.mid);
        push(L, off, p + "bn3.g", LP_KIND_BN_GAMMA, b.cout);
        push(L, off, p + "bn3.b", LP_KIND_BN_BETA, b.cout);
        if (b.proj) {
          push(L, off, p + "sc.w", LP_KIND_CONV_W, b.cout, 1, 1, b.cin);
          push(L, off, p + "bns.g", LP_KIND_BN_GAMMA, b.cout);
          push(L, off, p + "bns.b", LP_KIND_BN_BETA, b.cout);
        }
      } else if (post) {
        push(L, off, p + "conv1.w", LP_KIND_CONV_W, b.cout, 3, 3, b.cin);
        push(L, off, p + "bn1.g", LP_KIND_BN_GAMMA, b.cout);
        push(L, off, p + "bn1.b", LP_KIND_BN_BETA, b.cout);
        push(L, off, p + "conv2.w", LP_KIND_CONV_W, b.cout, 3, 3, b.cout);
        push(L, off, p + "bn2.g", LP_KIND_BN_GAMMA, b.cout);
        push(L, off, p + "bn2.b", LP_KIND_BN_BETA, b.cout);
        if (b.proj) {
          push(L, off, p + "sc.w", LP_KIND_CONV_W, b.cout, 1, 1, b.cin);
          push(L, off, p + "bns.g", LP_KIND_BN_GAMMA, b.cout);
          push(L, off, p + "bns.b", LP_KIND_BN_BETA, b.cout);
        }
      } else {
        push(L, off, p + "bn1.g", LP_KIND_BN_GAMMA, b.cin);
        push(L, off, p + "bn1.b", LP_KIND_BN_BETA, b.cin);
        push(L, off, p + "conv1.w", LP_KIND_CONV_W, b.cout, 3, 3, b.cin);
        push(L, off, p + "bn2.g", LP_KIND_BN_GAMMA, b.cout);
        push(L, off, p + "bn2.b", LP_KIND_BN_BETA, b.cout);
        push(L, off, p + "conv2.w", LP_KIND_CONV_W, b.cout, 3, 3, b.cout);
        if (b.proj) push(L, off, p + "sc.w", LP_KIND_CONV_W, b.cout, 1, 1, b.cin);
      }
    }
    if (k == K - 1) {
      const int c = blocks.back().cout;
      if (!post) {
        push(L, off, "head.bn.g", LP_KIND_BN_GAMMA, c);
        push(L, off, "head.bn.b", LP_KIND_BN_BETA, c);
      }
      push(L, off, "head.fc.w", LP_KIND_FC_W, d.num_classes, c);
      push(L, off, "head.fc.b", LP_KIND_FC_B, d.num_classes);
    }
    if (total) *total = off;
    return LP_OK;
  }
};

}  // namespace lp
