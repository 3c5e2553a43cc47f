"""A whole BERT encoder forward on the quantised path (Sec. 3 of the paper).

Every Embedding and FC layer is the quantised one (`q8_embedding`, `q8_linear`); Softmax, Layer
Normalization and the attention products stay in FP32 (`q8_attention`, `q8_add_layernorm`); GELU is
fused into FFN1's epilogue.  The model is the post-LayerNorm encoder of BERT with random-initialised
weights ~ N(0, 0.02), LayerNorm gamma 1 / beta 0, no attention mask and no dropout (inference on
full-length synthetic sequences).

This module only orchestrates calls into the C ABI; torch supplies device memory.
"""
from __future__ import annotations

from typing import Callable, Optional

import numpy as np
import torch

from . import binding as q8
from . import synth

LN_EPS = 1e-12
FC_NAMES = ("qkv", "attn_out", "ffn1", "ffn2")


class Q8BertEncoder:
    """Random-init quantised BERT encoder.  `dims` is e.g. synth.BERT_BASE (hidden, ffn, heads, layers, vocab,
    max_pos); `config` selects the seed family (BASE_SEED + 1000 * config + tensor index)."""

    def __init__(self, dims: dict, config: int, device="cuda", layers: Optional[int] = None, keep_fp32=False):
        self.H, self.F, self.heads = dims["hidden"], dims["ffn"], dims["heads"]
        self.L = dims["layers"] if layers is None else layers
        self.V, self.P = dims["vocab"], dims["max_pos"]
        if self.H != self.heads * 64:
            raise ValueError("head dimension must be 64")
        self.device = torch.device(device)
        self.config = config
        self.keep_fp32 = keep_fp32          # tests keep the seeded fp32 tensors to feed the CPU checker
        self.fp32 = {}

        def quantised(name, shape, sigma_seed):
            w = synth.normal(shape, synth.WEIGHT_SIGMA, synth.seed_for(config, sigma_seed))
            if keep_fp32:
                self.fp32[name] = w
            return q8.q8_quantize_weight(torch.from_numpy(w).to(self.device))

        def bias(name, n, seed):
            b = synth.bias(n, synth.seed_for(config, seed))
            if keep_fp32:
                self.fp32[name] = b
            return torch.from_numpy(b).to(self.device)

        self.word, self.S_word = quantised("word", (self.V, self.H), 100)
        self.pos, self.S_pos = quantised("pos", (self.P, self.H), 101)
        self.typ, self.S_typ = quantised("typ", (2, self.H), 102)
        self.layers = []
        for l in range(self.L):
            s0 = 200 + 20 * l
            lay = {}
            for i, (name, K, N, act) in enumerate(synth.fc_set(self.H, self.F)):
                Wq, S_w = quantised(f"W.{l}.{name}", (N, K), s0 + 2 * i)
                lay[name] = dict(Wq=Wq, S_w=S_w, b=bias(f"b.{l}.{name}", N, s0 + 2 * i + 1), act=act, K=K, N=N,
                                 state=q8.new_calibrate_state(self.device))
            self.layers.append(lay)
        self._bufs = None

    # ------------------------------------------------------------------ buffers
    def _buffers(self, T: int):
        if self._bufs is None or self._bufs["T"] != T:
            d, f32 = self.device, torch.float32
            e = lambda n: torch.empty((T, n), dtype=f32, device=d)
            self._bufs = dict(T=T, ew=e(self.H), ep=e(self.H), et=e(self.H), h=e(self.H), qkv=e(3 * self.H),
                              ctx=e(self.H), ao=e(self.H), h1=e(self.H), f=e(self.F), f2=e(self.H),
                              ws=q8.new_workspace(T, self.F, max(self.H, self.F), d),
                              status=torch.zeros(1, dtype=torch.int32, device=d))
        return self._bufs

    def memory_bytes_int8(self) -> int:
        n = self.word.numel() + self.pos.numel() + self.typ.numel()
        for lay in self.layers:
            n += sum(lay[k]["Wq"].numel() for k in FC_NAMES)
        return n

    # ------------------------------------------------------------------ forward
    def forward(self, ids: torch.Tensor, B: int, S: int, scales: str = "static", decay: float = 0.9999,
                hook: Optional[Callable] = None, debug: bool = False) -> torch.Tensor:
        """ids: int32 [B*S] on the device.  scales: "static" (Eq. 4 scales from earlier calibrate passes),
        "dynamic" (Sec. 4.1, per incoming tensor) or "calibrate" (dynamic forward that also feeds each
        quantiser's input to q8_calibrate).  hook(layer, name, X, Y, fc, S_x, Xq, acc) is called after every
        quantised FC; with debug=True, Xq / acc are that call's Int8 activation and Int32 accumulator copies."""
        T = B * S
        bf = self._buffers(T)
        pos_ids = torch.arange(S, dtype=torch.int32, device=self.device).repeat(B)
        typ_ids = torch.zeros(T, dtype=torch.int32, device=self.device)
        q8.q8_embedding(ids, self.word, self.S_word, out=bf["ew"], dev_status=bf["status"])
        q8.q8_embedding(pos_ids, self.pos, self.S_pos, out=bf["ep"], dev_status=bf["status"])
        q8.q8_embedding(typ_ids, self.typ, self.S_typ, out=bf["et"], dev_status=bf["status"])
        q8.q8_add_layernorm(bf["ew"], bf["ep"], bf["et"], eps=LN_EPS, out=bf["h"])

        def fc(l, name, X, Y):
            p = self.layers[l][name]
            if scales == "calibrate":
                q8.q8_calibrate(X, decay, p["state"])
            S_x = q8.calibrate_S_x(p["state"]) if scales == "static" else None
            Xq = acc = None
            if debug:
                if "dbg_xq" not in bf:
                    bf["dbg_xq"] = torch.empty(T * max(self.H, self.F), dtype=torch.int8, device=self.device)
                    bf["dbg_acc"] = torch.empty(T * max(3 * self.H, self.F), dtype=torch.int32, device=self.device)
                Xq = bf["dbg_xq"][: T * p["K"]].view(T, p["K"])
                acc = bf["dbg_acc"][: T * p["N"]].view(T, p["N"])
            q8.q8_linear(X, p["Wq"], p["S_w"], S_x, p["b"], p["act"], Y=Y, workspace=bf["ws"], dbg_Xq=Xq, dbg_acc=acc)
            if hook is not None:
                hook(l, name, X, Y, p, S_x if S_x is not None else bf["ws"][4:8].view(torch.float32), Xq, acc)

        for l in range(self.L):
            fc(l, "qkv", bf["h"], bf["qkv"])
            q8.q8_attention(bf["qkv"], B, S, self.heads, ctx=bf["ctx"])
            fc(l, "attn_out", bf["ctx"], bf["ao"])
            q8.q8_add_layernorm(bf["ao"], bf["h"], eps=LN_EPS, out=bf["h1"])
            fc(l, "ffn1", bf["h1"], bf["f"])
            fc(l, "ffn2", bf["f"], bf["f2"])
            q8.q8_add_layernorm(bf["f2"], bf["h1"], eps=LN_EPS, out=bf["h"])
        return bf["h"]

    def forward_fused(self, ids: torch.Tensor, B: int, S: int) -> torch.Tensor:
        """The same forward with static (Eq. 4) scales and every quantiser folded into the kernel that produces
        its input: LayerNorm and attention also emit Int8 at the consuming FC's scale, FFN1 emits only Int8 at
        FFN2's scale.  No stand-alone quantise pass is left and FFN1's fp32 output never reaches HBM.  The
        Int8 tensors are identical to those of forward(), so the result is bit-identical too."""
        T = B * S
        bf = self._buffers(T)
        if "hq" not in bf:
            i8 = lambda n: torch.empty((T, n), dtype=torch.int8, device=self.device)
            bf.update(hq=i8(self.H), ctxq=i8(self.H), h1q=i8(self.H), fq=i8(self.F))
        sx = lambda l, name: q8.calibrate_S_x(self.layers[l][name]["state"])
        pos_ids = torch.arange(S, dtype=torch.int32, device=self.device).repeat(B)
        typ_ids = torch.zeros(T, dtype=torch.int32, device=self.device)
        q8.q8_embedding(ids, self.word, self.S_word, out=bf["ew"], dev_status=bf["status"])
        q8.q8_embedding(pos_ids, self.pos, self.S_pos, out=bf["ep"], dev_status=bf["status"])
        q8.q8_embedding(typ_ids, self.typ, self.S_typ, out=bf["et"], dev_status=bf["status"])
        q8.q8_add_layernorm_quant(bf["ew"], bf["ep"], bf["et"], sx(0, "qkv"), out_q=bf["hq"], out=bf["h"], eps=LN_EPS)
        st = bf["status"]
        for l in range(self.L):
            p = self.layers[l]
            q8.q8_linear_q(bf["hq"], sx(l, "qkv"), p["qkv"]["Wq"], p["qkv"]["S_w"], p["qkv"]["b"], 0, Y=bf["qkv"],
                           dev_status=st)
            q8.q8_attention_quant(bf["qkv"], B, S, self.heads, sx(l, "attn_out"), ctx_q=bf["ctxq"])
            q8.q8_linear_q(bf["ctxq"], sx(l, "attn_out"), p["attn_out"]["Wq"], p["attn_out"]["S_w"], p["attn_out"]["b"],
                           0, Y=bf["ao"], dev_status=st)
            q8.q8_add_layernorm_quant(bf["ao"], bf["h"], None, sx(l, "ffn1"), out_q=bf["h1q"], out=bf["h1"], eps=LN_EPS)
            q8.q8_linear_q_requant(bf["h1q"], sx(l, "ffn1"), p["ffn1"]["Wq"], p["ffn1"]["S_w"], p["ffn1"]["b"], 1,
                                   sx(l, "ffn2"), Yq=bf["fq"], dev_status=st)
            q8.q8_linear_q(bf["fq"], sx(l, "ffn2"), p["ffn2"]["Wq"], p["ffn2"]["S_w"], p["ffn2"]["b"], 0, Y=bf["f2"],
                           dev_status=st)
            if l + 1 < self.L:
                q8.q8_add_layernorm_quant(bf["f2"], bf["h1"], None, sx(l + 1, "qkv"), out_q=bf["hq"], out=bf["h"],
                                          eps=LN_EPS)
            else:
                q8.q8_add_layernorm(bf["f2"], bf["h1"], eps=LN_EPS, out=bf["h"])
        return bf["h"]

    def forward_dynamic_fused(self, ids: torch.Tensor, B: int, S: int) -> torch.Tensor:
        """Dynamic quantisation (Sec. 4.1: every FC derives its scale from max|x| of the incoming tensor) without a
        single stand-alone abs-max pass: every kernel that produces an FC input (LayerNorm, attention, FFN1's
        epilogue) also folds max|output| into a device word, and the consuming FC takes 127 / that maximum.  Same
        Int8 tensors and the same result, bit for bit, as forward(scales="dynamic")."""
        T = B * S
        bf = self._buffers(T)
        if "amax" not in bf:
            bf["amax"] = torch.zeros(4 * self.L, dtype=torch.int32, device=self.device)
        amax = bf["amax"]
        amax.zero_()                      # the words only ever rise: start every forward at zero (one memset)
        word = lambda l, i: amax[4 * l + i: 4 * l + i + 1]
        pos_ids = torch.arange(S, dtype=torch.int32, device=self.device).repeat(B)
        typ_ids = torch.zeros(T, dtype=torch.int32, device=self.device)
        q8.q8_embedding(ids, self.word, self.S_word, out=bf["ew"], dev_status=bf["status"])
        q8.q8_embedding(pos_ids, self.pos, self.S_pos, out=bf["ep"], dev_status=bf["status"])
        q8.q8_embedding(typ_ids, self.typ, self.S_typ, out=bf["et"], dev_status=bf["status"])
        q8.q8_add_layernorm_absmax(bf["ew"], word(0, 0), bf["ep"], bf["et"], eps=LN_EPS, out=bf["h"])
        for l in range(self.L):
            p = self.layers[l]
            lin = lambda name, X, xw, Y, yw=None: q8.q8_linear_dyn(X, xw, p[name]["Wq"], p[name]["S_w"], p[name]["b"],
                                                                   p[name]["act"], Y=Y, y_absmax=yw, workspace=bf["ws"])
            lin("qkv", bf["h"], word(l, 0), bf["qkv"])
            q8.q8_attention_absmax(bf["qkv"], B, S, self.heads, word(l, 1), ctx=bf["ctx"])
            lin("attn_out", bf["ctx"], word(l, 1), bf["ao"])
            q8.q8_add_layernorm_absmax(bf["ao"], word(l, 2), bf["h"], eps=LN_EPS, out=bf["h1"])
            lin("ffn1", bf["h1"], word(l, 2), bf["f"], word(l, 3))
            lin("ffn2", bf["f"], word(l, 3), bf["f2"])
            if l + 1 < self.L:
                q8.q8_add_layernorm_absmax(bf["f2"], word(l + 1, 0), bf["h1"], eps=LN_EPS, out=bf["h"])
            else:
                q8.q8_add_layernorm(bf["f2"], bf["h1"], eps=LN_EPS, out=bf["h"])
        return bf["h"]

    def capture(self, ids: torch.Tensor, B: int, S: int, fused: bool = True):
        """Captures one static-scale forward into a CUDA graph (the forward is a fixed sequence of launches on
        fixed buffers, and for small batches the host cannot issue them as fast as the GPU runs them).
        Returns (graph, output tensor); graph.replay() recomputes the output from the current contents of `ids`."""
        run = (lambda: self.forward_fused(ids, B, S)) if fused else (lambda: self.forward(ids, B, S))
        run()                                   # first-call set-up (function attributes, buffers) outside capture
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            out = run()
        return graph, out

    def launches_per_forward(self, scales: str = "static", fused: bool = False) -> int:
        if fused and scales == "dynamic":
            return 4 + self.L * 11          # per layer: 4 x (quantise + GEMM), attention, two LayerNorms
        if fused:
            return 4 + self.L * 7
        per_fc = 2 if scales == "static" else (3 if scales == "dynamic" else 5)
        return 4 + self.L * (4 * per_fc + 3)

    def poll(self):
        """(code, bits) of the embedding status word and of the FC workspace, after synchronising."""
        a = q8.q8_poll_status(self._bufs["status"])
        b = q8.q8_poll_status(self._bufs["ws"])
        return a, b


def random_ids(count: int, vocab: int, config: int, device="cuda") -> torch.Tensor:
    return torch.from_numpy(synth.token_ids(count, vocab, synth.seed_for(config, 90))).to(device)
