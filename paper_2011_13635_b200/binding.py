"""ctypes binding of libmslt.so: argument marshalling only.

Every step of the training path runs in the library's CUDA kernels; torch is
used here for device memory, streams and nothing else.  Importing this module
loads the shared library and fails loudly if it has not been built
(`python -m paper_2011_13635_b200.build`).
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmslt.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2011_13635_b200.build`; "
                      "there is no fallback path")
lib = C.CDLL(LIB_PATH)


class Arch(C.Structure):
    _fields_ = [("hidden", C.c_int32), ("heads", C.c_int32), ("ffn", C.c_int32), ("vocab", C.c_int32),
                ("max_pos", C.c_int32), ("init_layers", C.c_int32), ("max_layers", C.c_int32),
                ("max_batch", C.c_int32), ("max_seq", C.c_int32), ("max_pred", C.c_int32),
                ("dtype", C.c_int32), ("ln_eps", C.c_float), ("max_trainable", C.c_int32),
                ("share_group", C.c_int32), ("nsp", C.c_int32)]


class Opt(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float), ("bias_correction", C.c_int32), ("lamb", C.c_int32)]


class GemmDesc(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("M", C.c_int32), ("N", C.c_int32), ("K", C.c_int32),
                ("batch", C.c_int32), ("hdiv", C.c_int32),
                ("A", C.c_void_p), ("a_rs", C.c_int64), ("a_ks", C.c_int64), ("a_bo", C.c_int64),
                ("a_bi", C.c_int64),
                ("B", C.c_void_p), ("b_rs", C.c_int64), ("b_ks", C.c_int64), ("b_bo", C.c_int64),
                ("b_bi", C.c_int64),
                ("D", C.c_void_p), ("ldd", C.c_int64), ("d_bo", C.c_int64), ("d_bi", C.c_int64),
                ("d_fp32", C.c_int32), ("accumulate", C.c_int32), ("alpha", C.c_float),
                ("bias", C.c_void_p), ("act", C.c_int32), ("aux", C.c_void_p),
                ("residual", C.c_void_p), ("split_k", C.c_int32), ("seq_lens", C.c_void_p)]


EXPORTS = ["mslt_query_bytes", "mslt_create", "mslt_destroy", "mslt_add_layers", "mslt_set_trainable",
           "mslt_set_optimizer", "mslt_step", "mslt_step_nsp", "mslt_step_backward", "mslt_step_apply", "mslt_num_grad_buckets",
           "mslt_grad_bucket", "mslt_set_bucket_hook", "mslt_read_loss", "mslt_forward", "mslt_num_layers",
           "mslt_num_trainable", "mslt_num_tensors", "mslt_tensor_info", "mslt_get_param",
           "mslt_set_param", "mslt_get_param_raw", "mslt_get_grad", "mslt_get_opt_state",
           "mslt_launch_count", "mslt_set_timing", "mslt_get_timings", "mslt_get_kernel_profile",
           "mslt_last_error",
           "mslt_op_gemm", "mslt_op_gemm_enqueue", "mslt_op_cross_entropy",
           "mslt_op_cross_entropy_scratch_bytes", "mslt_op_cross_entropy_noalloc", "mslt_op_layernorm",
           "mslt_op_layernorm_bwd", "mslt_op_softmax", "mslt_op_softmax_bwd", "mslt_op_colsum",
           "mslt_op_attention", "mslt_op_attention_bwd",
           "mslt_debug_starve_next_gemm", "mslt_debug_starve_next_attention", "mslt_debug_check_guards",
           "mslt_debug_set_gemm_variant"]

lib.mslt_last_error.restype = C.c_char_p
lib.mslt_last_error.argtypes = [C.c_void_p]
lib.mslt_launch_count.restype = C.c_int64
lib.mslt_launch_count.argtypes = [C.c_void_p]
lib.mslt_query_bytes.argtypes = [C.POINTER(Arch), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
lib.mslt_create.argtypes = [C.POINTER(Arch), C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t,
                            C.c_void_p, C.POINTER(C.c_void_p)]
lib.mslt_destroy.argtypes = [C.c_void_p]
BUCKET_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_int32)
lib.mslt_step_backward.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                   C.c_int32, C.c_void_p, C.POINTER(C.c_float)]
lib.mslt_step_apply.argtypes = [C.c_void_p]
lib.mslt_step_nsp.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                              C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_float)]
lib.mslt_num_grad_buckets.argtypes = [C.c_void_p]
lib.mslt_grad_bucket.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_void_p), C.POINTER(C.c_int64)]
lib.mslt_set_bucket_hook.argtypes = [C.c_void_p, C.c_void_p, BUCKET_FN, C.c_void_p]
lib.mslt_add_layers.argtypes = [C.c_void_p, C.c_int32]
lib.mslt_set_trainable.argtypes = [C.c_void_p, C.c_int32]
lib.mslt_set_optimizer.argtypes = [C.c_void_p, C.POINTER(Opt)]
lib.mslt_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                          C.c_int32, C.c_int32, C.POINTER(C.c_float)]
lib.mslt_read_loss.argtypes = [C.c_void_p, C.POINTER(C.c_float)]
lib.mslt_forward.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p,
                             C.c_void_p, C.c_int32, C.c_void_p]
lib.mslt_num_layers.argtypes = [C.c_void_p]
lib.mslt_num_trainable.argtypes = [C.c_void_p]
lib.mslt_num_tensors.argtypes = [C.c_void_p]
lib.mslt_tensor_info.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_char_p), C.POINTER(C.c_int32),
                                 C.POINTER(C.c_int64), C.POINTER(C.c_int32)]
lib.mslt_get_param.argtypes = [C.c_void_p, C.c_char_p, C.c_void_p, C.c_size_t]
lib.mslt_set_param.argtypes = [C.c_void_p, C.c_char_p, C.c_void_p, C.c_size_t]
lib.mslt_get_param_raw.argtypes = [C.c_void_p, C.c_char_p, C.c_void_p, C.c_size_t]
lib.mslt_get_grad.argtypes = [C.c_void_p, C.c_char_p, C.c_void_p, C.c_size_t]
lib.mslt_get_opt_state.argtypes = [C.c_void_p, C.c_char_p, C.c_int32, C.c_void_p, C.c_size_t]
lib.mslt_set_timing.argtypes = [C.c_void_p, C.c_int32]
lib.mslt_get_timings.argtypes = [C.c_void_p, C.c_void_p, C.c_int32]
lib.mslt_get_kernel_profile.argtypes = [C.c_void_p, C.c_void_p, C.c_int32]
lib.mslt_op_gemm.argtypes = [C.POINTER(GemmDesc), C.c_void_p, C.c_void_p]
lib.mslt_op_gemm_enqueue.argtypes = [C.POINTER(GemmDesc), C.c_void_p, C.c_void_p]


lib.mslt_op_cross_entropy_scratch_bytes.restype = C.c_size_t
lib.mslt_op_cross_entropy_scratch_bytes.argtypes = [C.c_int32]
lib.mslt_op_cross_entropy.argtypes = [C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_int32, C.c_int32,
                                      C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]


lib.mslt_op_cross_entropy_noalloc.argtypes = [C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_int32, C.c_int32,
                                              C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]


_P = C.c_void_p
lib.mslt_debug_starve_next_gemm.argtypes = [C.c_int32]
lib.mslt_debug_starve_next_attention.argtypes = [C.c_int32]
lib.mslt_debug_set_gemm_variant.argtypes = [C.c_int32]
lib.mslt_debug_check_guards.argtypes = [C.c_void_p, C.POINTER(C.c_int32)]
lib.mslt_op_layernorm.argtypes = [C.c_int32, _P, _P, _P, _P, _P, C.c_int32, C.c_int32, C.c_float, _P, C.c_int32]
lib.mslt_op_layernorm_bwd.argtypes = [C.c_int32, _P, _P, _P, _P, _P, _P, _P, _P, C.c_int32, C.c_int32, _P, C.c_int32]
lib.mslt_op_softmax.argtypes = [C.c_int32, _P, _P, _P, C.c_int32, C.c_int32, C.c_int32, C.c_float, _P, C.c_int32]
lib.mslt_op_softmax_bwd.argtypes = [C.c_int32, _P, _P, C.c_int32, C.c_int32, C.c_float, _P, C.c_int32]
lib.mslt_op_attention.argtypes = [_P, _P, _P, _P, C.c_int32, C.c_int32, C.c_int32, C.c_float, _P, _P, C.c_int32]
lib.mslt_op_attention_bwd.argtypes = [_P, _P, _P, _P, C.c_int32, C.c_int32, C.c_int32, C.c_float, _P, _P, C.c_int32]
lib.mslt_op_colsum.argtypes = [C.c_int32, _P, C.c_int64, C.c_int32, C.c_int32, _P, _P, C.c_int32]


class MsltError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"mslt error {code}: {msg}")
        self.code = code


def _check(rc: int):
    if rc != 0:
        raise MsltError(rc, (lib.mslt_last_error(None) or b"").decode())


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def mslt_query_bytes(arch: Arch):
    pb, wb = C.c_size_t(), C.c_size_t()
    _check(lib.mslt_query_bytes(C.byref(arch), C.byref(pb), C.byref(wb)))
    return pb.value, wb.value


def mslt_op_gemm(desc: GemmDesc, stream: int, status) -> None:
    _check(lib.mslt_op_gemm(C.byref(desc), C.c_void_p(stream), C.c_void_p(_ptr(status))))


def mslt_op_gemm_enqueue(desc: GemmDesc, stream: int, status) -> None:
    _check(lib.mslt_op_gemm_enqueue(C.byref(desc), C.c_void_p(stream), C.c_void_p(_ptr(status))))


def mslt_op_cross_entropy(dtype: int, logits, labels, V: int, dlogits, loss, scratch, stream: int) -> None:
    """logits fp32 [R, ldl], labels int32 [R], dlogits [R, ldd] or None, loss fp32 [1], scratch uint8:
    CUDA tensors."""
    R = logits.shape[0]
    _check(lib.mslt_op_cross_entropy(dtype, logits.data_ptr(), logits.stride(0), labels.data_ptr(), R, V,
                                     _ptr(dlogits), 0 if dlogits is None else dlogits.stride(0),
                                     loss.data_ptr(), scratch.data_ptr(), scratch.numel(), C.c_void_p(stream)))


def mslt_op_cross_entropy_noalloc(dtype: int, logits, labels, V: int, dlogits, loss, stream: int) -> None:
    """As mslt_op_cross_entropy, with the scratch taken from the library's built-in array (at most
    16384 rows; calls on one GPU must not overlap)."""
    R = logits.shape[0]
    _check(lib.mslt_op_cross_entropy_noalloc(dtype, logits.data_ptr(), logits.stride(0), labels.data_ptr(), R,
                                             V, _ptr(dlogits), 0 if dlogits is None else dlogits.stride(0),
                                             loss.data_ptr(), C.c_void_p(stream)))


def _dt(t) -> int:
    import torch
    return 1 if t.dtype == torch.bfloat16 else 0


def mslt_op_layernorm(z, gamma, beta, y, stats, eps: float, stream: int, sync: bool = True) -> None:
    """z, y [rows, H] float or bf16; gamma, beta fp32 [H]; stats fp32 [rows, 2] or None: CUDA tensors."""
    _check(lib.mslt_op_layernorm(_dt(z), z.data_ptr(), gamma.data_ptr(), beta.data_ptr(), y.data_ptr(),
                                 _ptr(stats), z.shape[0], z.shape[1], eps, C.c_void_p(stream), int(sync)))


def mslt_op_layernorm_bwd(dy, z, stats, gamma, dz, dgamma, dbeta, stream: int, sync: bool = True,
                          dbias=None) -> None:
    """dbias (fp32 [H] or None) receives += the column sums of dz."""
    _check(lib.mslt_op_layernorm_bwd(_dt(z), dy.data_ptr(), z.data_ptr(), stats.data_ptr(), gamma.data_ptr(),
                                     dz.data_ptr(), dgamma.data_ptr(), dbeta.data_ptr(), _ptr(dbias), z.shape[0],
                                     z.shape[1], C.c_void_p(stream), int(sync)))


def mslt_op_softmax(scores, probs, seq_lens, rows_per_seq: int, scale: float, stream: int,
                    sync: bool = True) -> None:
    """scores, probs [rows, S] (may be the same tensor); seq_lens int32 [rows / rows_per_seq] or None."""
    _check(lib.mslt_op_softmax(_dt(scores), scores.data_ptr(), probs.data_ptr(), _ptr(seq_lens),
                               scores.shape[0], scores.shape[1], rows_per_seq, scale, C.c_void_p(stream),
                               int(sync)))


def mslt_op_attention(qkv, probs, ctx, seq_lens, B: int, S: int, heads: int, scale: float, status,
                      stream: int, sync: bool = True) -> None:
    """qkv bf16 [B*S, 3*heads*64]; probs bf16 [B, heads, S, S] or None; ctx bf16 [B*S, heads*64]."""
    _check(lib.mslt_op_attention(qkv.data_ptr(), _ptr(probs), ctx.data_ptr(), _ptr(seq_lens), B, S, heads,
                                 scale, status.data_ptr(), C.c_void_p(stream), int(sync)))


def mslt_op_attention_bwd(qkv, probs, dctx, dqkv, B: int, S: int, heads: int, scale: float, status,
                          stream: int, sync: bool = True) -> None:
    """qkv, dqkv bf16 [B*S, 3*heads*64]; probs bf16 [B, heads, S, S]; dctx bf16 [B*S, heads*64]."""
    _check(lib.mslt_op_attention_bwd(qkv.data_ptr(), probs.data_ptr(), dctx.data_ptr(), dqkv.data_ptr(), B, S,
                                     heads, scale, status.data_ptr(), C.c_void_p(stream), int(sync)))


def mslt_op_softmax_bwd(dp, probs, scale: float, stream: int, sync: bool = True) -> None:
    _check(lib.mslt_op_softmax_bwd(_dt(dp), dp.data_ptr(), probs.data_ptr(), dp.shape[0], dp.shape[1], scale,
                                   C.c_void_p(stream), int(sync)))


def mslt_op_colsum(x, n: int, out, stream: int, sync: bool = True) -> None:
    """out[:n] += x[:, :n].sum(0); x [rows, ld] float or bf16, out fp32."""
    _check(lib.mslt_op_colsum(_dt(x), x.data_ptr(), x.stride(0), x.shape[0], n, out.data_ptr(),
                              C.c_void_p(stream), int(sync)))


class Mslt:
    """A stage-training context.  Device buffers are torch tensors owned by this object."""

    def __init__(self, *, hidden, heads, ffn, vocab, max_pos, init_layers, max_layers, max_batch,
                 max_seq, max_pred, dtype: str, ln_eps: float = 1e-12, max_trainable: int = 0,
                 share_group: int = 1, nsp: bool = False, device="cuda:0", stream=None):
        import torch
        self.torch = torch
        if not torch.cuda.is_available():
            raise MsltError(-4, "no CUDA device: this library has no CPU path")
        self.device = torch.device(device)
        self.arch = Arch(hidden, heads, ffn, vocab, max_pos, init_layers, max_layers, max_batch,
                         max_seq, max_pred, {"fp32": 0, "bf16": 1}[dtype], ln_eps, max_trainable, share_group, int(bool(nsp)))
        self.dtype = dtype
        pb, wb = mslt_query_bytes(self.arch)
        with torch.cuda.device(self.device):
            self._params = torch.empty(pb, dtype=torch.uint8, device=self.device)
            self._ws = torch.empty(wb, dtype=torch.uint8, device=self.device)
            self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
            h = C.c_void_p()
            _check(lib.mslt_create(C.byref(self.arch), self._params.data_ptr(), pb, self._ws.data_ptr(),
                                   wb, C.c_void_p(self.stream.cuda_stream), C.byref(h)))
        self.h = h
        self.param_bytes, self.workspace_bytes = pb, wb

    @classmethod
    def from_config(cls, cfg, *, init_layers=None, max_layers=None, **kw):
        return cls(hidden=cfg.hidden, heads=cfg.heads, ffn=cfg.ffn, vocab=cfg.vocab,
                   max_pos=cfg.max_pos, init_layers=cfg.layers if init_layers is None else init_layers,
                   max_layers=cfg.layers if max_layers is None else max_layers,
                   max_batch=cfg.batch, max_seq=cfg.seq, max_pred=cfg.pred, dtype=cfg.dtype,
                   share_group=getattr(cfg, "share_group", 1), nsp=getattr(cfg, "nsp", False), **kw)

    def close(self):
        if getattr(self, "h", None):
            lib.mslt_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()

    # -- staging ------------------------------------------------------------------------------
    def mslt_add_layers(self, k: int):
        _check(lib.mslt_add_layers(self.h, k))

    def mslt_set_trainable(self, top_k: int):
        _check(lib.mslt_set_trainable(self.h, top_k))

    def mslt_set_optimizer(self, lr, beta1=0.9, beta2=0.999, eps=1e-6, weight_decay=0.01,
                           bias_correction=1, lamb=0):
        o = Opt(lr, beta1, beta2, eps, weight_decay, int(bias_correction), int(lamb))
        _check(lib.mslt_set_optimizer(self.h, C.byref(o)))

    # -- the hot path -------------------------------------------------------------------------
    def mslt_step(self, tokens, seq_lens, mlm_positions, mlm_labels, sync: bool = True):
        """tokens [B,S], seq_lens [B] or None, positions/labels [B,P]: int32 CUDA tensors.
        Returns the loss (float) when sync, else None."""
        B, S = tokens.shape
        P = mlm_positions.shape[1]
        loss = C.c_float()
        _check(lib.mslt_step(self.h, tokens.data_ptr(), _ptr(seq_lens), mlm_positions.data_ptr(),
                             mlm_labels.data_ptr(), B, S, P, C.byref(loss) if sync else None))
        return loss.value if sync else None

    def mslt_step_nsp(self, tokens, seq_lens, segment_ids, mlm_positions, mlm_labels, nsp_labels, sync: bool = True):
        """The step with both objectives; segment_ids [B,S] and nsp_labels [B] int32 CUDA tensors or None."""
        B, S = tokens.shape
        P = mlm_positions.shape[1]
        loss = C.c_float()
        _check(lib.mslt_step_nsp(self.h, tokens.data_ptr(), _ptr(seq_lens), _ptr(segment_ids), mlm_positions.data_ptr(),
                                 mlm_labels.data_ptr(), _ptr(nsp_labels), B, S, P, C.byref(loss) if sync else None))
        return loss.value if sync else None

    def mslt_step_backward(self, tokens, seq_lens, mlm_positions, mlm_labels, total_valid=None, sync: bool = True):
        """Forward, loss and backward only; total_valid: int32 CUDA tensor of one element (valid slots
        over all workers) or None.  Returns this worker's share of the loss when sync."""
        B, S = tokens.shape
        P = mlm_positions.shape[1]
        loss = C.c_float()
        _check(lib.mslt_step_backward(self.h, tokens.data_ptr(), _ptr(seq_lens), mlm_positions.data_ptr(),
                                      mlm_labels.data_ptr(), B, S, P, _ptr(total_valid),
                                      C.byref(loss) if sync else None))
        return loss.value if sync else None

    def mslt_step_apply(self):
        _check(lib.mslt_step_apply(self.h))

    def grad_buckets(self):
        """The trainable gradients as float32 CUDA tensors that alias the gradient arena, in the order
        in which a backward pass completes them (output layer, layers top-down, embeddings)."""
        torch = self.torch
        flat = self._params.view(torch.float32)
        out = []
        for i in range(lib.mslt_num_grad_buckets(self.h)):
            ptr, cnt = C.c_void_p(), C.c_int64()
            _check(lib.mslt_grad_bucket(self.h, i, C.byref(ptr), C.byref(cnt)))
            first = (ptr.value - self._params.data_ptr()) // 4
            out.append(flat[first:first + cnt.value])
        return out

    def mslt_set_bucket_hook(self, comm_stream, fn):
        """fn(bucket_index) is called on the host when a bucket's kernels are enqueued; None clears."""
        if fn is None:
            self._hook = None
            _check(lib.mslt_set_bucket_hook(self.h, None, BUCKET_FN(), None))
            return
        self._hook = BUCKET_FN(lambda user, i: fn(int(i)))      # keep the callback object alive
        _check(lib.mslt_set_bucket_hook(self.h, C.c_void_p(comm_stream.cuda_stream), self._hook, None))

    def mslt_read_loss(self) -> float:
        loss = C.c_float()
        _check(lib.mslt_read_loss(self.h, C.byref(loss)))
        return loss.value

    def mslt_forward(self, tokens, seq_lens=None, mlm_positions=None, want_hidden=True):
        """Returns (hidden [B,S,H] in the compute dtype or None, logits [B*P,V] fp32 or None)."""
        torch = self.torch
        B, S = tokens.shape
        hidden = logits = None
        if want_hidden:
            hidden = torch.empty((B, S, self.arch.hidden), device=self.device,
                                 dtype=torch.bfloat16 if self.dtype == "bf16" else torch.float32)
        P = 0
        if mlm_positions is not None:
            P = mlm_positions.shape[1]
            logits = torch.empty((B * P, self.arch.vocab), device=self.device, dtype=torch.float32)
        _check(lib.mslt_forward(self.h, tokens.data_ptr(), _ptr(seq_lens), B, S, _ptr(hidden),
                                _ptr(mlm_positions), P, _ptr(logits)))
        return hidden, logits

    # -- inspection -----------------------------------------------------------------------------
    @property
    def num_layers(self) -> int:
        return lib.mslt_num_layers(self.h)

    @property
    def num_trainable(self) -> int:
        return lib.mslt_num_trainable(self.h)

    @property
    def launch_count(self) -> int:
        return lib.mslt_launch_count(self.h)

    def tensors(self) -> Dict[str, dict]:
        out = {}
        for i in range(lib.mslt_num_tensors(self.h)):
            name, rank, tr = C.c_char_p(), C.c_int32(), C.c_int32()
            shape = (C.c_int64 * 2)()
            _check(lib.mslt_tensor_info(self.h, i, C.byref(name), C.byref(rank), shape, C.byref(tr)))
            shp = (shape[0], shape[1]) if rank.value == 2 else (shape[0],)
            out[name.value.decode()] = dict(shape=shp, trainable=bool(tr.value))
        return out

    def _shape(self, name):
        info = self.tensors().get(name)
        return info["shape"] if info else (0,)   # unknown names are reported by the library

    def mslt_set_param(self, name: str, value: np.ndarray):
        v = np.ascontiguousarray(value, dtype=np.float32)
        _check(lib.mslt_set_param(self.h, name.encode(), v.ctypes.data, v.size))

    def set_params(self, weights: Dict[str, np.ndarray]):
        for k, v in weights.items():
            self.mslt_set_param(k, v)

    def mslt_get_param(self, name: str, shape=None) -> np.ndarray:
        shape = self._shape(name) if shape is None else shape
        out = np.empty(shape, dtype=np.float32)
        _check(lib.mslt_get_param(self.h, name.encode(), out.ctypes.data, out.size))
        return out

    def mslt_get_param_raw(self, name: str, shape=None) -> np.ndarray:
        shape = self._shape(name) if shape is None else shape
        two_byte = self.dtype == "bf16" and len(shape) == 2
        out = np.empty(shape, dtype=np.uint16 if two_byte else np.uint32)
        _check(lib.mslt_get_param_raw(self.h, name.encode(), out.ctypes.data, out.nbytes))
        return out

    def mslt_get_grad(self, name: str, shape=None) -> np.ndarray:
        shape = self._shape(name) if shape is None else shape
        out = np.empty(shape, dtype=np.float32)
        _check(lib.mslt_get_grad(self.h, name.encode(), out.ctypes.data, out.size))
        return out

    def mslt_get_opt_state(self, name: str, which: int, shape=None) -> np.ndarray:
        shape = self._shape(name) if shape is None else shape
        out = np.empty(shape, dtype=np.float32)
        _check(lib.mslt_get_opt_state(self.h, name.encode(), which, out.ctypes.data, out.size))
        return out

    def mslt_debug_check_guards(self) -> int:
        """Number of workspace guard bands that a kernel has written into (0 = none)."""
        bad = C.c_int32()
        _check(lib.mslt_debug_check_guards(self.h, C.byref(bad)))
        return bad.value

    def mslt_set_timing(self, level: int):
        _check(lib.mslt_set_timing(self.h, int(level)))

    PROFILE_CLASSES = ["linear", "attention", "ln_fwd", "ln_bwd", "softmax_fwd", "softmax_bwd", "colsum",
                       "cross_entropy", "adam", "other"]

    def mslt_get_kernel_profile(self) -> Dict[str, dict]:
        """Per kernel class: launches, work (flops for the two GEMM classes, bytes otherwise), ms."""
        buf = (C.c_double * 30)()
        _check(lib.mslt_get_kernel_profile(self.h, buf, 30))
        return {k: dict(launches=int(buf[3 * i]), work=buf[3 * i + 1], ms=buf[3 * i + 2])
                for i, k in enumerate(self.PROFILE_CLASSES)}

    def mslt_get_timings(self) -> Dict[str, float]:
        buf = (C.c_float * 5)()
        _check(lib.mslt_get_timings(self.h, buf, 5))
        return dict(zip(["frozen_fwd", "train_fwd", "head", "encoder_bwd", "adam"], list(buf)))
