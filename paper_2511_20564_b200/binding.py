"""ctypes binding of libe2egrec.so: argument marshalling only.

Every computation happens inside the library's CUDA kernels.  There is no CPU or
PyTorch fallback: if the shared library is missing or a call fails, an exception
is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libe2egrec.so")

F32, BF16 = 0, 1
ACCUMULATE_DW = 1
_DTYPES = {torch.float32: F32, torch.bfloat16: BF16}


class E2EGrecError(RuntimeError):
    pass


class Csr(C.Structure):
    _fields_ = [("n_nodes", C.c_int64), ("n_edges", C.c_int64), ("indptr", C.c_void_p),
                ("indices", C.c_void_p), ("edge_cum", C.c_void_p)]


class Mat(C.Structure):
    _fields_ = [("data", C.c_void_p), ("rows", C.c_int64), ("dim", C.c_int32), ("ld", C.c_int64),
                ("dtype", C.c_int32)]


class Block(C.Structure):
    _fields_ = [("cap_dst", C.c_int32), ("cap_src", C.c_int32), ("cap_edges", C.c_int32),
                ("counts", C.c_void_p), ("indptr", C.c_void_p), ("col", C.c_void_p),
                ("nbr_global", C.c_void_p), ("src_nodes", C.c_void_p), ("csc_ptr", C.c_void_p),
                ("csc_row", C.c_void_p), ("csc_eid", C.c_void_p), ("csc_col", C.c_void_p),
                ("inv_cnt", C.c_void_p)]


_lib = None


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_SO):
            raise E2EGrecError(f"{_SO} is missing: run `python -m paper_2511_20564_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(_SO)
        L.e2egrec_status_string.restype = C.c_char_p
        L.e2egrec_status_string.argtypes = [C.c_int32]
        L.e2egrec_last_error.restype = C.c_char_p
        L.e2egrec_sample_khop_workspace.restype = C.c_int32
        L.e2egrec_sample_khop_workspace.argtypes = [C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                                    C.c_void_p, C.c_void_p, C.POINTER(C.c_size_t)]
        L.e2egrec_sampler_scratch_init.restype = C.c_int32
        L.e2egrec_sampler_scratch_init.argtypes = [C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p]
        L.e2egrec_sampler_set_step.restype = C.c_int32
        L.e2egrec_sampler_set_step.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p]
        L.e2egrec_sample_join.restype = C.c_int32
        L.e2egrec_sample_join.argtypes = [C.c_void_p]
        L.e2egrec_blocks_transpose.restype = C.c_int32
        L.e2egrec_blocks_transpose.argtypes = [C.c_int64, C.c_int32, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.e2egrec_sample_khop.restype = C.c_int32
        L.e2egrec_sample_khop.argtypes = [C.POINTER(Csr), C.c_void_p, C.c_int32, C.c_int32, C.c_void_p,
                                          C.c_uint64, C.c_uint32, C.c_uint32, C.POINTER(Block), C.c_void_p,
                                          C.c_size_t, C.c_void_p]
        L.e2egrec_lightgcn_sampled_forward.restype = C.c_int32
        L.e2egrec_lightgcn_sampled_forward.argtypes = [C.POINTER(Block), C.c_int32, C.POINTER(Mat), C.c_void_p, C.c_void_p,
                                                       C.POINTER(C.c_size_t), C.POINTER(Mat), C.c_void_p]
        L.e2egrec_lightgcn_sampled_backward.restype = C.c_int32
        L.e2egrec_lightgcn_sampled_backward.argtypes = [C.POINTER(Block), C.c_int32, C.c_void_p, C.POINTER(Mat),
                                                        C.POINTER(Mat), C.c_void_p, C.POINTER(C.c_size_t), C.c_void_p]
        L.e2egrec_ssl_loss.restype = C.c_int32
        L.e2egrec_ssl_loss.argtypes = [C.POINTER(Mat), C.POINTER(Mat), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                       C.POINTER(Mat), C.c_void_p, C.POINTER(C.c_size_t), C.c_void_p]
        L.e2egrec_gradient_norm.restype = C.c_int32
        L.e2egrec_gradient_norm.argtypes = [C.POINTER(Mat), C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(C.c_size_t),
                                            C.c_void_p]
        L.e2egrec_gradient_norms.restype = C.c_int32
        L.e2egrec_gradient_norms.argtypes = [C.POINTER(Mat), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                             C.POINTER(C.c_size_t), C.c_void_p]
        L.e2egrec_gradnorm_update.restype = C.c_int32
        L.e2egrec_gradnorm_update.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_float,
                                              C.c_float, C.c_void_p, C.c_void_p]
        L.e2egrec_gate_fusion_forward.restype = C.c_int32
        L.e2egrec_gate_fusion_forward.argtypes = [C.POINTER(Mat), C.c_int32, C.POINTER(Mat), C.c_void_p, C.POINTER(Mat),
                                                  C.POINTER(Mat), C.c_void_p, C.POINTER(C.c_size_t), C.c_void_p]
        L.e2egrec_gate_fusion_backward.restype = C.c_int32
        L.e2egrec_gate_fusion_backward.argtypes = [C.POINTER(Mat), C.POINTER(Mat), C.c_int32, C.POINTER(Mat), C.POINTER(Mat),
                                                   C.POINTER(Mat), C.c_void_p, C.c_void_p, C.c_void_p,
                                                   C.POINTER(C.c_size_t), C.c_void_p]
        L.e2egrec_edge_cumulate.restype = C.c_int32
        L.e2egrec_edge_cumulate.argtypes = [C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.e2egrec_sage_forward.restype = C.c_int32
        L.e2egrec_sage_forward.argtypes = [C.POINTER(Block), C.c_int32, C.POINTER(Mat), C.POINTER(Mat),
                                           C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(C.c_size_t),
                                           C.POINTER(Mat), C.c_void_p]
        L.e2egrec_sage_backward.restype = C.c_int32
        L.e2egrec_sage_backward.argtypes = [C.POINTER(Block), C.c_int32, C.POINTER(Mat), C.POINTER(Mat),
                                            C.c_void_p, C.c_void_p, C.POINTER(Mat), C.c_void_p, C.c_void_p,
                                            C.POINTER(Mat), C.c_void_p, C.POINTER(C.c_size_t), C.c_uint32,
                                            C.c_void_p]
        L.e2egrec_sage_backward_multi.restype = C.c_int32
        L.e2egrec_sage_backward_multi.argtypes = [C.POINTER(Block), C.c_int32, C.POINTER(Mat), C.POINTER(Mat),
                                                  C.c_void_p, C.c_void_p, C.POINTER(Mat), C.c_int32, C.c_void_p, C.c_void_p,
                                                  C.POINTER(Mat), C.c_void_p, C.POINTER(C.c_size_t), C.c_uint32,
                                                  C.c_void_p]
        L.e2egrec_sage_ctx_layout.restype = C.c_int32
        L.e2egrec_sage_ctx_layout.argtypes = [C.POINTER(Block), C.c_int32, C.POINTER(Mat), C.POINTER(Mat),
                                              C.c_void_p, C.c_void_p, C.c_void_p]
        L.e2egrec_aggregate_forward.restype = C.c_int32
        L.e2egrec_aggregate_forward.argtypes = [C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.POINTER(Mat),
                                                C.POINTER(Mat), C.c_uint32, C.c_void_p, C.POINTER(C.c_size_t),
                                                C.c_void_p]
        L.e2egrec_aggregate_backward.restype = C.c_int32
        L.e2egrec_aggregate_backward.argtypes = [C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                                 C.POINTER(Mat), C.POINTER(Mat), C.c_void_p, C.POINTER(C.c_size_t),
                                                 C.c_void_p]
        L.e2egrec_aggregate_forward_static.restype = C.c_int32
        L.e2egrec_aggregate_forward_static.argtypes = [C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.POINTER(Mat),
                                                       C.POINTER(Mat), C.c_uint32, C.c_void_p]
        L.e2egrec_aggregate_forward_static_limit.restype = C.c_size_t
        L.e2egrec_joint_step.restype = C.c_int32
        L.e2egrec_joint_step.argtypes = [C.POINTER(Csr), C.POINTER(Mat), C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                         C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.POINTER(Mat), C.POINTER(Mat),
                                         C.c_void_p, C.c_uint64, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_void_p, C.POINTER(Mat), C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.POINTER(C.c_size_t), C.c_void_p]
        L.e2egrec_joint_step_phase.restype = C.c_int32
        L.e2egrec_joint_step_phase.argtypes = L.e2egrec_joint_step.argtypes[:-1] + [C.c_uint32, C.c_void_p]
        L.e2egrec_joint_step_layout.restype = C.c_int32
        L.e2egrec_joint_step_layout.argtypes = [C.POINTER(Csr), C.POINTER(Mat), C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                                C.POINTER(Mat), C.POINTER(Mat), C.c_uint32, C.c_void_p, C.c_void_p,
                                                C.c_void_p, C.c_void_p, C.c_void_p]
        L.e2egrec_graph_from_coo.restype = C.c_int32
        L.e2egrec_graph_from_coo.argtypes = [C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.c_void_p, C.POINTER(C.c_size_t), C.c_void_p]
        L.e2egrec_csr_transpose.restype = C.c_int32
        L.e2egrec_csr_transpose.argtypes = [C.POINTER(Csr), C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.POINTER(C.c_size_t), C.c_void_p]
        for fn in (L.e2egrec_lightgcn_forward, L.e2egrec_lightgcn_backward):
            fn.restype = C.c_int32
            fn.argtypes = [C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(Mat),
                           C.POINTER(Mat), C.c_void_p, C.POINTER(C.c_size_t), C.c_void_p]
        L.e2egrec_launch_count.restype = C.c_uint64
        L.e2egrec_profile_tap.restype = C.c_int32
        L.e2egrec_profile_tap.argtypes = [C.c_int32, C.c_void_p, C.c_void_p]
        _lib = L
    return _lib


def launch_count() -> int:
    return int(lib().e2egrec_launch_count())


def profile_tap(which: int, start_event=None, stop_event=None):
    """Arms the timing tap `which` with two torch.cuda.Event(enable_timing=True) that have been recorded
    at least once (so that their CUDA handles exist); see e2egrec_profile_tap."""
    a = None if start_event is None else C.c_void_p(start_event.cuda_event)
    b = None if stop_event is None else C.c_void_p(stop_event.cuda_event)
    _check(lib().e2egrec_profile_tap(which, a, b), "e2egrec_profile_tap")


def status_string(code: int) -> str:
    return lib().e2egrec_status_string(code).decode()


def _check(rc: int, what: str):
    if rc != 0:
        extra = lib().e2egrec_last_error().decode() if rc in (-7, -5) else ""
        raise E2EGrecError(f"{what}: {status_string(rc)} ({rc}) {extra}".strip())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _mat(t: torch.Tensor) -> Mat:
    assert t.dim() == 2 and t.stride(1) == 1
    return Mat(t.data_ptr(), t.shape[0], t.shape[1], t.stride(0), _DTYPES[t.dtype])


def _i32_host(values):
    return (C.c_int32 * len(values))(*[int(v) for v in values])


def _dev_bytes(n: int, device):
    """256-byte aligned device buffer of at least n bytes (torch's allocator aligns to 512)."""
    return torch.empty(max(int(n), 256), dtype=torch.uint8, device=device)


# ------------------------------------------------------------------------------------------ sampling

def sample_khop_workspace(n_nodes: int, n_seeds: int, fanouts):
    """-> (cap_dst[], cap_src[], cap_edges[], scratch_bytes)"""
    L = len(fanouts)
    f = _i32_host(fanouts)
    cd, cs, ce = (C.c_int32 * L)(), (C.c_int32 * L)(), (C.c_int32 * L)()
    nbytes = C.c_size_t(0)
    _check(lib().e2egrec_sample_khop_workspace(n_nodes, n_seeds, L, f, cd, cs, ce, C.byref(nbytes)),
           "e2egrec_sample_khop_workspace")
    return list(cd), list(cs), list(ce), nbytes.value


class Blocks:
    """Device buffers for the blocks of one k-hop sample, sized for the worst case."""

    def __init__(self, n_nodes: int, n_seeds: int, fanouts, device="cuda"):
        self.fanouts = [int(f) for f in fanouts]
        self.n_nodes, self.n_seeds = int(n_nodes), int(n_seeds)
        cd, cs, ce, self.scratch_bytes = sample_khop_workspace(n_nodes, n_seeds, self.fanouts)
        self.caps = list(zip(cd, cs, ce))
        self.t = []
        i32 = dict(dtype=torch.int32, device=device)
        self.counts = torch.zeros(len(self.caps), 4, **i32)    # row h: {n_dst, n_src, n_edges, status} of hop h+1
        for h, (d, s, e) in enumerate(self.caps):
            self.t.append(dict(
                counts=self.counts[h], indptr=torch.zeros(d + 1, **i32), col=torch.zeros(max(e, 1), **i32),
                nbr_global=torch.zeros(max(e, 1), **i32), src_nodes=torch.zeros(max(s, 1), **i32),
                csc_ptr=torch.zeros(s + 1, **i32), csc_row=torch.zeros(max(e, 1), **i32),
                csc_eid=torch.zeros(max(e, 1), **i32), csc_col=torch.zeros(max(e, 1), **i32),
                inv_cnt=torch.zeros(max(d, 1), dtype=torch.float32, device=device)))
        self.c = (Block * len(self.caps))()
        for h, ((d, s, e), t) in enumerate(zip(self.caps, self.t)):
            self.c[h] = Block(d, s, e, *[t[k].data_ptr() for k in
                                         ("counts", "indptr", "col", "nbr_global", "src_nodes", "csc_ptr",
                                          "csc_row", "csc_eid", "csc_col", "inv_cnt")])
        self.scratch = _dev_bytes(self.scratch_bytes, device)
        sampler_scratch_init(n_nodes, self.scratch)

    def __len__(self):
        return len(self.caps)

    def to_host(self):
        """Copies the blocks back, trimmed to their true sizes (synchronises)."""
        out = []
        for t in self.t:
            n_dst, n_src, n_edges, status = t["counts"].tolist()
            out.append(dict(n_dst=n_dst, n_src=n_src, n_edges=n_edges, status=status,
                            indptr=t["indptr"][: n_dst + 1].cpu().numpy(), col=t["col"][:n_edges].cpu().numpy(),
                            nbr_global=t["nbr_global"][:n_edges].cpu().numpy(),
                            src_nodes=t["src_nodes"][:n_src].cpu().numpy(),
                            csc_ptr=t["csc_ptr"][: n_src + 1].cpu().numpy(),
                            csc_row=t["csc_row"][:n_edges].cpu().numpy(),
                            csc_eid=t["csc_eid"][:n_edges].cpu().numpy(),
                            csc_col=t["csc_col"][:n_edges].cpu().numpy(),
                            inv_cnt=t["inv_cnt"][:n_dst].cpu().numpy()))
        return out


def sampler_scratch_init(n_nodes: int, scratch: torch.Tensor, stream=None):
    _check(lib().e2egrec_sampler_scratch_init(n_nodes, _ptr(scratch), scratch.numel(), _stream(stream)),
           "e2egrec_sampler_scratch_init")


def sampler_set_step(scratch: torch.Tensor, step_offset: int, stream=None):
    _check(lib().e2egrec_sampler_set_step(_ptr(scratch), step_offset & 0xFFFFFFFF, _stream(stream)),
           "e2egrec_sampler_set_step")


DEFER_TRANSPOSE = 1
NO_TRANSPOSE = 2


def sample_join(stream=None):
    _check(lib().e2egrec_sample_join(_stream(stream)), "e2egrec_sample_join")


def edge_cumulate(indptr: torch.Tensor, q: torch.Tensor, stream=None):
    """Per-row running sums (uint64, returned as an int64 tensor of the same bits) of the integer edge weights q
    (uint32 values in an int32 / uint32 tensor); see e2egrec_edge_cumulate."""
    assert indptr.dtype == torch.int64 and q.element_size() == 4 and q.is_contiguous()
    cum = torch.empty(max(q.numel(), 1), dtype=torch.int64, device=q.device)
    _check(lib().e2egrec_edge_cumulate(indptr.numel() - 1, q.numel(), _ptr(indptr), _ptr(q), _ptr(cum), _stream(stream)),
           "e2egrec_edge_cumulate")
    return cum[: q.numel()]


def sample_khop(indptr: torch.Tensor, indices: torch.Tensor, seeds: torch.Tensor, blocks: Blocks, seed: int,
                step: int, stream=None, defer_transpose=False, edge_cum=None, transpose=True):
    """Enqueues the k-hop sample of `seeds` into `blocks` (see e2egrec_sample_khop); edge_cum (from edge_cumulate)
    switches to the weighted draws; transpose=False leaves the transposed form to blocks_transpose."""
    assert indptr.dtype == torch.int64 and indices.dtype == torch.int32 and seeds.dtype == torch.int32
    assert edge_cum is None or (edge_cum.element_size() == 8 and edge_cum.numel() == indices.numel())
    g = Csr(indptr.numel() - 1, indices.numel(), indptr.data_ptr(), indices.data_ptr(),
            None if edge_cum is None else edge_cum.data_ptr())
    f = _i32_host(blocks.fanouts)
    _check(lib().e2egrec_sample_khop(C.byref(g), _ptr(seeds), seeds.numel(), len(blocks), f,
                                     C.c_uint64(seed), C.c_uint32(step),
                                     (DEFER_TRANSPOSE if defer_transpose else 0) | (0 if transpose else NO_TRANSPOSE), blocks.c,
                                     _ptr(blocks.scratch),
                                     blocks.scratch.numel(), _stream(stream)), "e2egrec_sample_khop")


def blocks_transpose(blocks: Blocks, stream=None):
    """Builds the transposed form of blocks sampled with transpose=False (see e2egrec_blocks_transpose)."""
    _check(lib().e2egrec_blocks_transpose(C.c_int64(blocks.n_nodes), len(blocks), blocks.c, _ptr(blocks.scratch),
                                          C.c_size_t(blocks.scratch.numel()), _stream(stream)), "e2egrec_blocks_transpose")


# ------------------------------------------------------------------------------------------ GraphSAGE

def _mats(ts):
    arr = (Mat * len(ts))()
    for i, t in enumerate(ts):
        arr[i] = _mat(t)
    return arr


def _ptr_array(ts, n):
    if ts is None:
        return None
    arr = (C.c_void_p * n)()
    for i, t in enumerate(ts):
        arr[i] = None if t is None else t.data_ptr()
    return arr


def sage_forward_ctx_bytes(blocks: Blocks, X, Ws) -> int:
    n = C.c_size_t(0)
    x, w = _mat(X), _mats(Ws)
    _check(lib().e2egrec_sage_forward(blocks.c, len(Ws), C.byref(x), w, None, None, None, C.byref(n), None, None),
           "e2egrec_sage_forward(size query)")
    return n.value


def sage_forward(blocks: Blocks, X, Ws, biases=None, acts=None, ctx=None, H_out=None, stream=None):
    """Enqueues the forward pass; returns (H_out, ctx).  ctx / H_out are allocated when not given."""
    L = len(Ws)
    if ctx is None:
        ctx = _dev_bytes(sage_forward_ctx_bytes(blocks, X, Ws), X.device)
    if H_out is None:
        H_out = torch.zeros(max(blocks.caps[0][0], 1), Ws[-1].shape[0], dtype=X.dtype, device=X.device)
    x, w, ho = _mat(X), _mats(Ws), _mat(H_out)
    n = C.c_size_t(ctx.numel())
    a = None if acts is None else _i32_host(acts)
    _check(lib().e2egrec_sage_forward(blocks.c, L, C.byref(x), w, _ptr_array(biases, L), a, _ptr(ctx), C.byref(n),
                                      C.byref(ho), _stream(stream)), "e2egrec_sage_forward")
    return H_out, ctx


def sage_ctx_views(blocks: Blocks, X, Ws, ctx):
    """Views into ctx: per layer (cat [rows x 2 d_in], h_out [rows x d_out]); see e2egrec_sage_ctx_layout."""
    L = len(Ws)
    co, ho, rows = (C.c_size_t * L)(), (C.c_size_t * L)(), (C.c_int64 * L)()
    x, w = _mat(X), _mats(Ws)
    _check(lib().e2egrec_sage_ctx_layout(blocks.c, L, C.byref(x), w, co, ho, rows), "e2egrec_sage_ctx_layout")
    es = X.element_size()
    out = []
    for l, W in enumerate(Ws):
        r, d_out, k = rows[l], W.shape[0], W.shape[1]
        cat = ctx[co[l]: co[l] + r * k * es].view(X.dtype).view(r, k)
        h = ctx[ho[l]: ho[l] + r * d_out * es].view(X.dtype).view(r, d_out)
        out.append((cat, h))
    return out


def sage_backward_scratch_bytes(blocks: Blocks, X, Ws) -> int:
    n = C.c_size_t(0)
    x, w = _mat(X), _mats(Ws)
    _check(lib().e2egrec_sage_backward(blocks.c, len(Ws), C.byref(x), w, None, None, None, None, None, None, None,
                                       C.byref(n), 0, None), "e2egrec_sage_backward(size query)")
    return n.value


def sage_backward(blocks: Blocks, X, Ws, ctx, dH_out, acts=None, dWs=None, dbs=None, dX_rows=None, scratch=None,
                  accumulate=False, stream=None):
    """Enqueues the backward pass; returns (dWs, dX_rows).  Buffers are allocated when not given."""
    L = len(Ws)
    dev = X.device
    if scratch is None:
        scratch = _dev_bytes(sage_backward_scratch_bytes(blocks, X, Ws), dev)
    if dWs is None:
        dWs = [torch.zeros(W.shape, dtype=torch.float32, device=dev) for W in Ws]
    if dX_rows is None:
        dX_rows = torch.zeros(max(blocks.caps[L - 1][1], 1), X.shape[1], dtype=X.dtype, device=dev)
    x, w, dh, dx = _mat(X), _mats(Ws), _mat(dH_out), _mat(dX_rows)
    n = C.c_size_t(scratch.numel())
    a = None if acts is None else _i32_host(acts)
    _check(lib().e2egrec_sage_backward(blocks.c, L, C.byref(x), w, a, _ptr(ctx), C.byref(dh), _ptr_array(dWs, L),
                                       _ptr_array(dbs, L), C.byref(dx), _ptr(scratch), C.byref(n),
                                       ACCUMULATE_DW if accumulate else 0, _stream(stream)), "e2egrec_sage_backward")
    return dWs, dX_rows


def sage_backward_multi_scratch_bytes(blocks: Blocks, X, Ws, n_rhs: int) -> int:
    n = C.c_size_t(0)
    x, w = _mat(X), _mats(Ws)
    _check(lib().e2egrec_sage_backward_multi(blocks.c, len(Ws), C.byref(x), w, None, None, None, n_rhs, None, None, None, None,
                                             C.byref(n), 0, None), "e2egrec_sage_backward_multi(size query)")
    return n.value


def sage_backward_multi(blocks: Blocks, X, Ws, ctx, dH_outs, acts=None, dWs=None, dbs=None, dX_rows=None, scratch=None,
                        accumulate=False, stream=None):
    """Enqueues one backward pass for the gradients in the list dH_outs (one or two); returns (dWs, list of dX_rows):
    dWs is the sum over the gradients, dX_rows[r] belongs to dH_outs[r].  Buffers are allocated when not given."""
    L, R = len(Ws), len(dH_outs)
    dev = X.device
    if scratch is None:
        scratch = _dev_bytes(sage_backward_multi_scratch_bytes(blocks, X, Ws, R), dev)
    if dWs is None:
        dWs = [torch.zeros(W.shape, dtype=torch.float32, device=dev) for W in Ws]
    if dX_rows is None:
        dX_rows = [torch.zeros(max(blocks.caps[L - 1][1], 1), X.shape[1], dtype=X.dtype, device=dev) for _ in range(R)]
    x, w = _mat(X), _mats(Ws)
    dh, dx = _mats(dH_outs), _mats(dX_rows)
    n = C.c_size_t(scratch.numel())
    a = None if acts is None else _i32_host(acts)
    _check(lib().e2egrec_sage_backward_multi(blocks.c, L, C.byref(x), w, a, _ptr(ctx), dh, R, _ptr_array(dWs, L),
                                             _ptr_array(dbs, L), dx, _ptr(scratch), C.byref(n),
                                             ACCUMULATE_DW if accumulate else 0, _stream(stream)), "e2egrec_sage_backward_multi")
    return dWs, dX_rows


# ------------------------------------------------------------------------------------------ whole graph

def aggregate_ws_bytes(n_entries, X) -> int:
    """Scratch bytes e2egrec_aggregate_forward asks for with n_entries entries and rows like X's (size query only)."""
    x = _mat(X)
    n = C.c_size_t(0)
    _check(lib().e2egrec_aggregate_forward(1, int(n_entries), None, None, C.byref(x), C.byref(x), 0, None, C.byref(n), None),
           "e2egrec_aggregate_forward(size query)")
    return n.value


def aggregate_forward(indptr, indices, X, out=None, ws=None, sum_only=False, stream=None):
    """Enqueues out[i] = mean (or sum) of X[indices[row i]]; returns (out, ws)."""
    n_dst, n_entries = indptr.numel() - 1, indices.numel()
    if out is None:
        out = torch.empty(max(n_dst, 1), X.shape[1], dtype=X.dtype, device=X.device)
    x, o = _mat(X), _mat(out)
    n = C.c_size_t(0)
    if ws is None:
        _check(lib().e2egrec_aggregate_forward(n_dst, n_entries, None, None, C.byref(x), C.byref(o), 0, None,
                                               C.byref(n), None), "e2egrec_aggregate_forward(size query)")
        ws = _dev_bytes(n.value, X.device)
    n = C.c_size_t(ws.numel())
    _check(lib().e2egrec_aggregate_forward(n_dst, n_entries, _ptr(indptr), _ptr(indices), C.byref(x), C.byref(o),
                                           1 if sum_only else 0, _ptr(ws), C.byref(n), _stream(stream)),
           "e2egrec_aggregate_forward")
    return out, ws


def aggregate_backward(csc_ptr, csc_row, inv_deg, G, dX=None, ws=None, stream=None):
    """Enqueues dX[s] = sum over column s of inv_deg[r] * G[r]; returns (dX, ws)."""
    n_src, n_entries = csc_ptr.numel() - 1, csc_row.numel()
    if dX is None:
        dX = torch.empty(max(n_src, 1), G.shape[1], dtype=G.dtype, device=G.device)
    g, o = _mat(G), _mat(dX)
    n = C.c_size_t(0)
    if ws is None:
        _check(lib().e2egrec_aggregate_backward(n_src, n_entries, None, None, None, C.byref(g), C.byref(o), None,
                                                C.byref(n), None), "e2egrec_aggregate_backward(size query)")
        ws = _dev_bytes(n.value, G.device)
    n = C.c_size_t(ws.numel())
    _check(lib().e2egrec_aggregate_backward(n_src, n_entries, _ptr(csc_ptr), _ptr(csc_row), _ptr(inv_deg),
                                            C.byref(g), C.byref(o), _ptr(ws), C.byref(n), _stream(stream)),
           "e2egrec_aggregate_backward")
    return dX, ws


def aggregate_forward_static(indptr, indices, X, out, sum_only=False, stream=None):
    """e2egrec_aggregate_forward_static: the same aggregation for callers that may not allocate device
    memory where they aggregate (they run inside someone else's memory pool, or at a point where an
    allocation would stall the GPU).  The scratch is a fixed 8 MiB buffer inside the library, so `out`
    must be supplied and nothing is allocated here; inputs that need more scratch raise E2EGrecError.
    Calls on one GPU share that buffer and must not overlap."""
    n_dst, n_entries = indptr.numel() - 1, indices.numel()
    x, o = _mat(X), _mat(out)
    _check(lib().e2egrec_aggregate_forward_static(n_dst, n_entries, _ptr(indptr), _ptr(indices), C.byref(x),
                                                  C.byref(o), 1 if sum_only else 0, _stream(stream)),
           "e2egrec_aggregate_forward_static")
    return out


def aggregate_forward_static_limit() -> int:
    return int(lib().e2egrec_aggregate_forward_static_limit())


# ------------------------------------------------------------------------------------------ joint step

JOINT_LINEAR = 0x100
JOINT_GATE = 0x200


class JointStep:
    """Buffers and arguments of e2egrec_joint_step for a fixed problem shape; `run` enqueues one step.

    linear=True: identity activations everywhere (E2EGREC_JOINT_LINEAR).  W_gate (and b_gate) given: the gating fusion
    of the concatenated features (E2EGREC_JOINT_GATE); they travel as the fourth entry of the tower's arrays, and their
    gradients come back as dW_tower[3], db_tower[3]."""

    def __init__(self, indptr, indices, X, n_pairs, dense_dim, fanouts, W_gnn, W_tower, b_tower=None, linear=False,
                 W_gate=None, b_gate=None):
        dev = X.device
        self.indptr, self.indices, self.X = indptr, indices, X
        self.n_nodes = indptr.numel() - 1
        self.n_pairs, self.dense_dim = int(n_pairs), int(dense_dim)
        self.fanouts = [int(f) for f in fanouts]
        self.W_gnn, self.W_tower = list(W_gnn), list(W_tower)[:3]
        self.b_tower = None if b_tower is None else list(b_tower)[:3]
        self.flags = (JOINT_LINEAR if linear else 0) | (JOINT_GATE if W_gate is not None else 0)
        if W_gate is not None:
            self.W_tower.append(W_gate)
            if self.b_tower is not None or b_gate is not None:
                self.b_tower = (self.b_tower or [None, None, None]) + [b_gate]
        self.n_tower = len(self.W_tower)
        L = len(self.fanouts)
        _, cs, _, _ = sample_khop_workspace(self.n_nodes, 2 * self.n_pairs, self.fanouts)
        self.cap_rows = max(cs[L - 1], 1)
        f32 = dict(dtype=torch.float32, device=dev)
        self.loss = torch.zeros(1, **f32)
        self.logits = torch.zeros(self.n_pairs, **f32)
        self.dW_gnn = [torch.zeros(W.shape, **f32) for W in self.W_gnn]
        self.dW_tower = [torch.zeros(W.shape, **f32) for W in self.W_tower]
        self.db_tower = [torch.zeros(W.shape[0], **f32) for W in self.W_tower]
        self.dX_rows = torch.zeros(self.cap_rows, X.shape[1], dtype=X.dtype, device=dev)
        self.dX_ids = torch.zeros(self.cap_rows, dtype=torch.int32, device=dev)
        self.n_rows = torch.zeros(2, dtype=torch.int32, device=dev)
        self._g = Csr(self.n_nodes, indices.numel(), indptr.data_ptr(), indices.data_ptr(), None)
        self._x, self._wg, self._wt, self._dx = _mat(X), _mats(self.W_gnn), _mats(self.W_tower), _mat(self.dX_rows)
        self._f = _i32_host(self.fanouts)
        n = C.c_size_t(0)
        self._call(None, None, None, None, n, None, 0, 0)
        self.ws = _dev_bytes(n.value, dev)
        sampler_scratch_init(self.n_nodes, self.ws)

    def _call(self, user, item, dense, labels, nbytes, stream, seed, step, phase=0):
        L, nt = len(self.fanouts), self.n_tower
        _check(lib().e2egrec_joint_step_phase(
            C.byref(self._g), C.byref(self._x), _ptr(user), _ptr(item), self.n_pairs, _ptr(dense), self.dense_dim,
            _ptr(labels), L, self._f, self._wg, self._wt, _ptr_array(self.b_tower, nt), C.c_uint64(seed),
            C.c_uint32(step), _ptr(self.loss), _ptr(self.logits), _ptr_array(self.dW_gnn, L),
            _ptr_array(self.dW_tower, nt), _ptr_array(self.db_tower, nt), C.byref(self._dx), _ptr(self.dX_ids),
            _ptr(self.n_rows), None if user is None else _ptr(self.ws), C.byref(nbytes), C.c_uint32(phase | self.flags),
            stream), "e2egrec_joint_step_phase")

    def run(self, pair_user, pair_item, dense, labels, seed, step, stream=None, phase=0):
        """phase 0: the whole step; 1: seeds + sampling only; 2: everything else, on the blocks phase 1 left in ws."""
        self._call(pair_user, pair_item, dense, labels, C.c_size_t(self.ws.numel()), _stream(stream), seed, step, phase)
        return self

    def activations(self):
        """Views into ws of what the last step left there (e2egrec_joint_step_layout): dict with the tower's z, a1, a2,
        gate, z_fused ([pair_rows x width]), `enc`, the list of encoder layer outputs ([rows x d_out]), and `counts`,
        the int32[4] counts of every hop's block."""
        L = len(self.fanouts)
        tower, enc, rows, prow = (C.c_size_t * 5)(), (C.c_size_t * L)(), (C.c_int64 * L)(), C.c_int64(0)
        cnt = (C.c_size_t * L)()
        _check(lib().e2egrec_joint_step_layout(C.byref(self._g), C.byref(self._x), self.n_pairs, self.dense_dim, L, self._f,
                                               self._wg, self._wt, C.c_uint32(self.flags), tower, enc, rows, C.byref(prow), cnt),
               "e2egrec_joint_step_layout")
        es, dt = self.X.element_size(), self.X.dtype
        zdim, h1, h2 = self.W_tower[0].shape[1], self.W_tower[0].shape[0], self.W_tower[1].shape[0]

        def view(off, r, c):
            return self.ws[off: off + r * c * es].view(dt).view(r, c)

        out = {k: view(tower[i], prow.value, w) for i, (k, w) in
               enumerate((("z", zdim), ("a1", h1), ("a2", h2), ("gate", zdim), ("z_fused", zdim)))}
        out["enc"] = [view(enc[l], rows[l], self.W_gnn[l].shape[0]) for l in range(L)]
        out["counts"] = [self.ws[cnt[h]: cnt[h] + 16].view(torch.int32) for h in range(L)]   # {n_dst, n_src, n_edges, status}
        return out


# ------------------------------------------------------------------------------------------ graph ingest

def graph_from_coo(n_nodes: int, row: torch.Tensor, col: torch.Tensor, stream=None):
    """Enqueues the canonical CSR of an edge list; returns (indptr int64, indices int32, status int32[1])."""
    m, dev = row.numel(), row.device
    indptr = torch.empty(n_nodes + 1, dtype=torch.int64, device=dev)
    indices = torch.empty(max(m, 1), dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    n = C.c_size_t(0)
    _check(lib().e2egrec_graph_from_coo(n_nodes, m, None, None, None, None, None, None, C.byref(n), None),
           "e2egrec_graph_from_coo(size query)")
    ws = _dev_bytes(n.value, dev)
    n = C.c_size_t(ws.numel())
    _check(lib().e2egrec_graph_from_coo(n_nodes, m, _ptr(row), _ptr(col), _ptr(indptr), _ptr(indices), _ptr(status),
                                        _ptr(ws), C.byref(n), _stream(stream)), "e2egrec_graph_from_coo")
    return indptr, indices[:m], status


def csr_transpose(indptr: torch.Tensor, indices: torch.Tensor, n_cols: int, stream=None):
    """Enqueues the CSC of a CSR; returns (csc_ptr int64, csc_row int32, csc_eid int64, status)."""
    m, dev = indices.numel(), indptr.device
    g = Csr(indptr.numel() - 1, m, indptr.data_ptr(), indices.data_ptr(), None)
    csc_ptr = torch.empty(n_cols + 1, dtype=torch.int64, device=dev)
    csc_row = torch.empty(max(m, 1), dtype=torch.int32, device=dev)
    csc_eid = torch.empty(max(m, 1), dtype=torch.int64, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    n = C.c_size_t(0)
    _check(lib().e2egrec_csr_transpose(C.byref(g), n_cols, None, None, None, None, None, C.byref(n), None),
           "e2egrec_csr_transpose(size query)")
    ws = _dev_bytes(n.value, dev)
    n = C.c_size_t(ws.numel())
    _check(lib().e2egrec_csr_transpose(C.byref(g), n_cols, _ptr(csc_ptr), _ptr(csc_row), _ptr(csc_eid), _ptr(status),
                                       _ptr(ws), C.byref(n), _stream(stream)), "e2egrec_csr_transpose")
    return csc_ptr, csc_row[:m], csc_eid[:m], status


# ------------------------------------------------------------------------------------------ LightGCN

def _lightgcn(fn, name, ptr, idx, inv_sqrt_deg, n_layers, Hin, out, ws, stream):
    n, m = ptr.numel() - 1, idx.numel()
    if out is None:
        out = torch.empty_like(Hin)
    a, b = _mat(Hin), _mat(out)
    nbytes = C.c_size_t(0)
    if ws is None:
        _check(fn(n, m, None, None, None, n_layers, C.byref(a), C.byref(b), None, C.byref(nbytes), None), name + "(size query)")
        ws = _dev_bytes(nbytes.value, Hin.device)
    nbytes = C.c_size_t(ws.numel())
    _check(fn(n, m, _ptr(ptr), _ptr(idx), _ptr(inv_sqrt_deg), n_layers, C.byref(a), C.byref(b), _ptr(ws), C.byref(nbytes),
              _stream(stream)), name)
    return out, ws


def lightgcn_forward(indptr, indices, inv_sqrt_deg, n_layers, H0, Y=None, ws=None, stream=None):
    """Enqueues Y = mean over layers of A_hat^l H0; returns (Y, ws)."""
    return _lightgcn(lib().e2egrec_lightgcn_forward, "e2egrec_lightgcn_forward", indptr, indices, inv_sqrt_deg, n_layers,
                     H0, Y, ws, stream)


def lightgcn_backward(csc_ptr, csc_row, inv_sqrt_deg, n_layers, dY, dH0=None, ws=None, stream=None):
    """Enqueues the adjoint of lightgcn_forward over the CSC arrays; returns (dH0, ws)."""
    return _lightgcn(lib().e2egrec_lightgcn_backward, "e2egrec_lightgcn_backward", csc_ptr, csc_row, inv_sqrt_deg,
                     n_layers, dY, dH0, ws, stream)


def lightgcn_sampled_forward(blocks: Blocks, X: torch.Tensor, inv_sqrt_deg: torch.Tensor, ctx=None, Y=None, stream=None):
    """Enqueues LightGCN on the sampled blocks (see e2egrec_lightgcn_sampled_forward); returns (Y, ctx)."""
    assert inv_sqrt_deg.dtype == torch.float32
    x = _mat(X)
    n = C.c_size_t(0)
    _check(lib().e2egrec_lightgcn_sampled_forward(blocks.c, len(blocks), C.byref(x), None, None, C.byref(n), None, None),
           "e2egrec_lightgcn_sampled_forward(size query)")
    if ctx is None:
        ctx = _dev_bytes(n.value, X.device)
    if Y is None:
        Y = torch.zeros(blocks.caps[0][0], X.shape[1], dtype=X.dtype, device=X.device)
    y = _mat(Y)
    n = C.c_size_t(ctx.numel())
    _check(lib().e2egrec_lightgcn_sampled_forward(blocks.c, len(blocks), C.byref(x), _ptr(inv_sqrt_deg), _ptr(ctx), C.byref(n),
                                                  C.byref(y), _stream(stream)), "e2egrec_lightgcn_sampled_forward")
    return Y, ctx


def lightgcn_sampled_backward(blocks: Blocks, ctx: torch.Tensor, dY: torch.Tensor, dX_rows=None, scratch=None, stream=None):
    """Enqueues the adjoint (see e2egrec_lightgcn_sampled_backward); returns (dX_rows, scratch)."""
    dy = _mat(dY)
    n = C.c_size_t(0)
    _check(lib().e2egrec_lightgcn_sampled_backward(blocks.c, len(blocks), None, C.byref(dy), None, None, C.byref(n), None),
           "e2egrec_lightgcn_sampled_backward(size query)")
    if scratch is None:
        scratch = _dev_bytes(n.value, dY.device)
    if dX_rows is None:
        dX_rows = torch.zeros(blocks.caps[-1][1], dY.shape[1], dtype=dY.dtype, device=dY.device)
    dx = _mat(dX_rows)
    n = C.c_size_t(scratch.numel())
    _check(lib().e2egrec_lightgcn_sampled_backward(blocks.c, len(blocks), _ptr(ctx), C.byref(dy), C.byref(dx), _ptr(scratch),
                                                   C.byref(n), _stream(stream)), "e2egrec_lightgcn_sampled_backward")
    return dX_rows, scratch


# ------------------------------------------------------------------------------------------ SSL task, GradNorm

_SUM_WS = {}


def _sum_ws(device):
    """The scratch of the fixed-order sums (size from the library's query), one per device."""
    key = str(device)
    if key not in _SUM_WS:
        n = C.c_size_t(0)
        _check(lib().e2egrec_gradient_norms(None, 1, None, None, None, C.byref(n), None), "e2egrec_gradient_norms(size query)")
        _SUM_WS[key] = _dev_bytes(n.value, device)
    return _SUM_WS[key]


def ssl_loss(H: torch.Tensor, X: torch.Tensor, seed_ids: torch.Tensor, n_rows_dev, weight: torch.Tensor, loss=None,
             dH=None, stream=None):
    """Enqueues L_ssl = ||X[seed_ids] - H||_F^2 and dH = 2 weight (H - X[seed_ids]); returns (loss, dH)."""
    assert weight.dtype == torch.float32 and seed_ids.dtype == torch.int32
    if loss is None:
        loss = torch.zeros(1, dtype=torch.float32, device=H.device)
    if dH is None:
        dH = torch.zeros_like(H)
    ws = _sum_ws(H.device)
    n = C.c_size_t(ws.numel())
    h, x, g = _mat(H), _mat(X), _mat(dH)
    _check(lib().e2egrec_ssl_loss(C.byref(h), C.byref(x), _ptr(seed_ids), None if n_rows_dev is None else _ptr(n_rows_dev),
                                  _ptr(weight), _ptr(loss), C.byref(g), _ptr(ws), C.byref(n), _stream(stream)),
           "e2egrec_ssl_loss")
    return loss, dH


def gradient_norm(A: torch.Tensor, n_rows_dev=None, out=None, stream=None):
    """Enqueues ||A[:n_rows]||_2 into a device float; see e2egrec_gradient_norm."""
    if out is None:
        out = torch.zeros(1, dtype=torch.float32, device=A.device)
    ws = _sum_ws(A.device)
    n = C.c_size_t(ws.numel())
    a = _mat(A)
    _check(lib().e2egrec_gradient_norm(C.byref(a), None if n_rows_dev is None else _ptr(n_rows_dev), _ptr(out), _ptr(ws),
                                       C.byref(n), _stream(stream)), "e2egrec_gradient_norm")
    return out


def gradient_norms(As, n_rows_dev=None, out=None, stream=None):
    """Enqueues the norms ||A[:n_rows]||_2 of up to four matrices of one shape into out[len(As)]; see e2egrec_gradient_norms."""
    if out is None:
        out = torch.zeros(len(As), dtype=torch.float32, device=As[0].device)
    ws = _sum_ws(As[0].device)
    n = C.c_size_t(ws.numel())
    _check(lib().e2egrec_gradient_norms(_mats(As), len(As), None if n_rows_dev is None else _ptr(n_rows_dev), _ptr(out), _ptr(ws),
                                        C.byref(n), _stream(stream)), "e2egrec_gradient_norms")
    return out


def gradnorm_update(w: torch.Tensor, L: torch.Tensor, L0: torch.Tensor, g: torch.Tensor, gamma=1.0, lr=0.025, L_gn=None,
                    stream=None):
    """Enqueues one GradNorm step on the device-resident task weights w (in place); see e2egrec_gradnorm_update."""
    for t in (w, L, L0, g):
        assert t.dtype == torch.float32 and t.numel() == w.numel()
    _check(lib().e2egrec_gradnorm_update(_ptr(w), _ptr(L), _ptr(L0), _ptr(g), w.numel(), C.c_float(gamma), C.c_float(lr),
                                         None if L_gn is None else _ptr(L_gn), _stream(stream)), "e2egrec_gradnorm_update")
    return w


# ------------------------------------------------------------------------------------------ gated fusion

def gate_fusion_forward(F: torch.Tensor, n_rows: int, Wg: torch.Tensor, bg=None, ws=None, stream=None):
    """Enqueues g = sigmoid(F Wg^T + bg), fused = g * F on the first n_rows rows; returns (fused, gate, ws)."""
    f, w = _mat(F), _mat(Wg)
    gate, fused = torch.zeros_like(F), torch.zeros_like(F)
    g, o = _mat(gate), _mat(fused)
    n = C.c_size_t(0)
    _check(lib().e2egrec_gate_fusion_forward(C.byref(f), n_rows, C.byref(w), None, None, None, None, C.byref(n), None),
           "e2egrec_gate_fusion_forward(size query)")
    if ws is None:
        ws = _dev_bytes(n.value, F.device)
    n = C.c_size_t(ws.numel())
    _check(lib().e2egrec_gate_fusion_forward(C.byref(f), n_rows, C.byref(w), _ptr(bg), C.byref(g), C.byref(o), _ptr(ws),
                                             C.byref(n), _stream(stream)), "e2egrec_gate_fusion_forward")
    return fused, gate, ws


def gate_fusion_backward(dFused: torch.Tensor, F: torch.Tensor, n_rows: int, gate: torch.Tensor, Wg: torch.Tensor, ws,
                         with_bias=True, stream=None):
    """Enqueues the adjoint of gate_fusion_forward; returns (dF, dWg, dbg)."""
    d = F.shape[1]
    dF = torch.zeros_like(F)
    dWg = torch.zeros(d, d, dtype=torch.float32, device=F.device)
    dbg = torch.zeros(d, dtype=torch.float32, device=F.device) if with_bias else None
    a, f, g, w, o = _mat(dFused), _mat(F), _mat(gate), _mat(Wg), _mat(dF)
    n = C.c_size_t(ws.numel())
    _check(lib().e2egrec_gate_fusion_backward(C.byref(a), C.byref(f), n_rows, C.byref(g), C.byref(w), C.byref(o), _ptr(dWg),
                                              _ptr(dbg), _ptr(ws), C.byref(n), _stream(stream)), "e2egrec_gate_fusion_backward")
    return dF, dWg, dbg
