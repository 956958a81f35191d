"""ctypes binding over libepara.so: the same names as the C ABI, argument marshalling only.

Every step of the path runs inside the library's CUDA kernels.  torch is used for device
memory and streams.  There is no fallback: if the library is missing, importing raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libepara.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it first (python -m paper_2511_00603_b200.build); "
                      "there is no CPU or eager fallback")
lib = C.CDLL(LIB_PATH)

OK, PENDING = 0, 1
E_INVALID, E_UNSUPPORTED, E_TIMEOUT, E_RESOURCE, E_DEVICE, E_CUDA = -1, -2, -3, -4, -5, -6
CAT_LS, CAT_FS, CAT_LS_GT1, CAT_FS_GT1 = 0, 1, 2, 3
MODEL_MLP, MODEL_VIT, MODEL_DECODER = 0, 1, 2
GEMM_TCGEN05, GEMM_SIMT, GEMM_TCGEN05_UNFUSED = 0, 1, 2
EPI_BIAS, EPI_GELU, EPI_SWIGLU, EPI_RESID_F32 = 1, 2, 4, 8
K_NAMES = ["gather", "norm", "gemm", "rope", "attn_dec", "attn_combine", "attn_enc", "assemble", "output", "gemm_stream", "trace", "attn_prefill"]
ERR_PAGE_APPEND, ERR_PAGE_ATTEND, ERR_SELFTEST_WAIT = 101, 102, 90
DECODE_STATUS_OFFSET = 192
K_COUNT = len(K_NAMES)


class Config(C.Structure):
    _fields_ = [("device", C.c_int), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
                ("cap_ls", C.c_int), ("cap_fs", C.c_int), ("mf_max", C.c_int), ("gemm_impl", C.c_int),
                ("max_queue", C.c_int), ("profile", C.c_int)]


class ModelDesc(C.Structure):
    _fields_ = [("kind", C.c_int), ("n_layers", C.c_int), ("d", C.c_int), ("n_heads", C.c_int),
                ("n_kv_heads", C.c_int), ("head_dim", C.c_int), ("ffn", C.c_int), ("vocab", C.c_int),
                ("img", C.c_int), ("patch", C.c_int), ("mlp_dims", C.POINTER(C.c_int)),
                ("tensors", C.POINTER(C.c_void_p)), ("n_tensors", C.c_int), ("kv_pool", C.c_void_p),
                ("kv_pages", C.c_longlong), ("max_kv_len", C.c_int), ("max_batch", C.c_int), ("trace", C.c_void_p)]


class Inputs(C.Structure):
    _fields_ = [("input", C.c_void_p), ("token", C.c_int), ("kv_len", C.c_int), ("block_table", C.c_void_p),
                ("n_blocks", C.c_int), ("tokens", C.POINTER(C.c_int32)), ("n_tokens", C.c_int), ("deadline_ns", C.c_longlong), ("arrival_ns", C.c_longlong),
                ("stream", C.c_int), ("out_logits", C.c_void_p), ("out_argmax", C.c_void_p)]


class StepInfo(C.Structure):
    _fields_ = [("step_id", C.c_uint64), ("admitted", C.c_int * 2), ("dropped", C.c_int * 2),
                ("launches", C.c_int), ("gemm_groups", C.c_int), ("gemm_flops", C.c_double),
                ("weight_bytes", C.c_double), ("kv_bytes", C.c_double), ("stream_gemm_flops", C.c_double),
                ("stream_weight_bytes", C.c_double), ("prefill_tokens", C.c_int)]


class Output(C.Structure):
    _fields_ = [("status", C.c_int), ("step_id", C.c_uint64), ("logits", C.c_void_p), ("n_out", C.c_int),
                ("argmax", C.c_void_p), ("device_error", C.c_int)]


class GemmProblem(C.Structure):
    _fields_ = [("A", C.c_void_p), ("W", C.c_void_p), ("C", C.c_void_p), ("bias", C.c_void_p),
                ("M", C.c_int), ("N", C.c_int), ("K", C.c_int), ("lda", C.c_int), ("ldw", C.c_int),
                ("ldc", C.c_int), ("epilogue", C.c_int)]


EXPORTS = ["epara_init", "epara_register_model", "epara_submit", "epara_submit_many", "epara_step", "epara_collect",
           "epara_step_profile", "epara_set_profile", "epara_destroy", "epara_strerror", "epara_model_workspace_bytes",
           "epara_dp_group_count", "epara_inter_request_count", "epara_admit_queue", "epara_grouped_gemm",
           "epara_gemm_scratch_bytes", "epara_gemm_scratch_bytes_for", "epara_decode_attention", "epara_decode_attention_scratch_bytes",
           "epara_decode_attention_static", "epara_static_scratch_bytes", "epara_decode_attention_static_status",
           "epara_set_max_profile_launches", "epara_selftest_bounded_wait", "epara_offload_probabilities", "epara_simulate",
           "epara_place_sssp"]

lib.epara_init.argtypes = [C.POINTER(Config), C.POINTER(C.c_void_p)]
lib.epara_register_model.argtypes = [C.c_void_p, C.POINTER(ModelDesc), C.POINTER(C.c_int)]
lib.epara_submit.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(Inputs), C.POINTER(C.c_uint64)]
lib.epara_submit_many.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(Inputs), C.c_int, C.POINTER(C.c_uint64),
                                  C.POINTER(C.c_int)]
lib.epara_step.argtypes = [C.c_void_p, C.c_void_p, C.c_longlong, C.POINTER(StepInfo)]
lib.epara_collect.argtypes = [C.c_void_p, C.c_uint64, C.POINTER(Output)]
lib.epara_step_profile.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.POINTER(C.c_int)]
lib.epara_set_profile.argtypes = [C.c_void_p, C.c_int]
lib.epara_destroy.argtypes = [C.c_void_p]
lib.epara_strerror.argtypes = [C.c_int]
lib.epara_strerror.restype = C.c_char_p
lib.epara_model_workspace_bytes.argtypes = [C.POINTER(Config), C.POINTER(ModelDesc)]
lib.epara_model_workspace_bytes.restype = C.c_size_t
lib.epara_dp_group_count.argtypes = [C.c_double, C.c_double]
lib.epara_inter_request_count.argtypes = [C.c_int, C.c_int]
lib.epara_admit_queue.argtypes = [C.c_int, C.POINTER(C.c_uint64), C.POINTER(C.c_longlong), C.POINTER(C.c_int),
                                  C.c_longlong, C.c_int, C.c_int, C.POINTER(C.c_uint64), C.POINTER(C.c_int),
                                  C.POINTER(C.c_uint64), C.POINTER(C.c_int)]
lib.epara_grouped_gemm.argtypes = [C.c_int, C.c_void_p, C.c_int, C.POINTER(GemmProblem), C.c_int, C.c_void_p,
                                   C.c_size_t]
lib.epara_gemm_scratch_bytes.argtypes = [C.c_int]
lib.epara_gemm_scratch_bytes.restype = C.c_size_t
lib.epara_gemm_scratch_bytes_for.argtypes = [C.c_int, C.POINTER(GemmProblem), C.c_int]
lib.epara_gemm_scratch_bytes_for.restype = C.c_size_t
lib.epara_decode_attention.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_longlong, C.c_void_p,
                                       C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int,
                                       C.c_int, C.c_void_p, C.c_size_t]
lib.epara_decode_attention_scratch_bytes.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int]
lib.epara_decode_attention_scratch_bytes.restype = C.c_size_t


lib.epara_decode_attention_static.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_longlong,
                                              C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                              C.c_int, C.c_int]
lib.epara_decode_attention_static_status.argtypes = [C.c_int, C.POINTER(C.c_int)]
lib.epara_set_max_profile_launches.argtypes = [C.c_void_p, C.c_int]
lib.epara_selftest_bounded_wait.argtypes = [C.c_int, C.c_void_p, C.c_ulonglong, C.c_void_p, C.POINTER(C.c_int)]
lib.epara_static_scratch_bytes.argtypes = []
lib.epara_static_scratch_bytes.restype = C.c_size_t


PROFILE_POINTS, MAX_OFFLOAD_DRAWS = 10, 5


class Cluster(C.Structure):
    _fields_ = [("n_servers", C.c_int), ("gpus", C.POINTER(C.c_int)), ("vram", C.c_double), ("sync_ms", C.c_double),
                ("offload_ms", C.c_double)]


class Service(C.Structure):
    _fields_ = [("a", C.c_double), ("b", C.c_double), ("n_gpus", C.c_int), ("cat", C.c_int), ("bs", C.c_int),
                ("slo_ms", C.c_double), ("fps", C.c_double), ("frames", C.c_int), ("c_ms", C.c_double * PROFILE_POINTS)]


class SimRequest(C.Structure):
    _fields_ = [("t_ms", C.c_double), ("service", C.c_int), ("server", C.c_int), ("u", C.c_double * MAX_OFFLOAD_DRAWS)]


class Placement(C.Structure):
    _fields_ = [("service", C.c_int), ("server", C.c_int)]


class SimResult(C.Structure):
    _fields_ = [("phi", C.c_double), ("served", C.c_int), ("timeout", C.c_int), ("offload_exceed", C.c_int),
                ("insufficient", C.c_int), ("late", C.c_int), ("offloads", C.c_int), ("instances", C.c_int)]


lib.epara_offload_probabilities.argtypes = [C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_double),
                                            C.POINTER(C.c_double), C.c_double, C.POINTER(C.c_double)]
lib.epara_simulate.argtypes = [C.POINTER(Cluster), C.POINTER(Service), C.c_int, C.POINTER(SimRequest), C.c_int,
                               C.POINTER(Placement), C.c_int, C.c_int, C.POINTER(SimResult)]
lib.epara_place_sssp.argtypes = [C.POINTER(Cluster), C.POINTER(Service), C.c_int, C.POINTER(SimRequest), C.c_int,
                                 C.POINTER(Placement), C.c_int, C.c_int, C.POINTER(Placement), C.c_int, C.POINTER(C.c_int)]


class EparaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib.epara_strerror(status).decode()} ({status})")


def _check(status: int, where: str) -> int:
    if status < 0:
        raise EparaError(status, where)
    return status


# ----------------------------------------------------------------------------- host policy
def epara_dp_group_count(required_fps: float, group_fps: float) -> int:
    return lib.epara_dp_group_count(required_fps, group_fps)


def epara_inter_request_count(bs: int, mf_max: int) -> int:
    return lib.epara_inter_request_count(bs, mf_max)


def epara_admit_queue(tickets: Sequence[int], deadlines: Sequence[int], streams: Sequence[int], now_ns: int,
                      cap: int, mf_max: int = 0):
    n = len(tickets)
    tk = (C.c_uint64 * max(n, 1))(*tickets)
    dl = (C.c_longlong * max(n, 1))(*deadlines)
    sd = (C.c_int * max(n, 1))(*streams)
    oa, od = (C.c_uint64 * max(n, 1))(), (C.c_uint64 * max(n, 1))()
    na, nd = C.c_int(), C.c_int()
    _check(lib.epara_admit_queue(n, tk, dl, sd, now_ns, cap, mf_max, oa, C.byref(na), od, C.byref(nd)),
           "epara_admit_queue")
    return list(oa[:na.value]), list(od[:nd.value])


# ----------------------------------------------------------------------------- model descriptors
def model_tensors(p: Dict) -> List:
    """Flat tensor list of a synth model in the order the C ABI documents (decoder layers must
    already be packed with synth.pack_decoder_layer)."""
    k = p["kind"]
    if k == "mlp":
        out = []
        for w, b in zip(p["W"], p["b"]):
            out += [w, b]
        return out
    if k == "vit":
        out = [p["W_pe"], p["b_pe"], p["cls"], p["pos"]]
        for L in p["layers"]:
            out += [L[n] for n in ("ln1_g", "ln1_b", "Wqkv", "bqkv", "Wo", "bo", "ln2_g", "ln2_b", "W1", "b1", "W2", "b2")]
        return out + [p["lnf_g"], p["lnf_b"], p["Whead"], p["bhead"]]
    if k == "decoder":
        out = [p["Emb"]]
        for L in p["packed_layers"]:
            out += [L[n] for n in ("g1", "Wqkv", "Wo", "g2", "Wgu", "Wd")]
        return out + [p["gf"], p["Wlm"]]
    raise ValueError(k)


def make_model_desc(p: Dict, kv_pool=None, max_kv_len: int = 0, max_batch: int = 0, kv_pages: int = 0, trace=None):
    """Returns (ModelDesc, keepalive) for a synth model whose tensors live on the device.
    kv_pages: pages per layer the library may touch (default: all of kv_pool's)."""
    tensors = model_tensors(p)
    for t in tensors:
        assert t.is_cuda and t.is_contiguous()
    arr = (C.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])
    d = ModelDesc()
    keep = [arr, tensors]
    d.tensors = C.cast(arr, C.POINTER(C.c_void_p))
    d.n_tensors = len(tensors)
    d.max_batch = max_batch
    if p["kind"] == "mlp":
        dims = (C.c_int * len(p["dims"]))(*p["dims"])
        keep.append(dims)
        d.kind, d.n_layers, d.mlp_dims = MODEL_MLP, len(p["dims"]) - 1, C.cast(dims, C.POINTER(C.c_int))
    elif p["kind"] == "vit":
        d.kind, d.n_layers, d.d, d.n_heads = MODEL_VIT, p["n_layers"], p["d"], p["n_heads"]
        d.head_dim, d.ffn, d.vocab, d.img, d.patch = p["d"] // p["n_heads"], p["mlp"], p["n_cls"], p["img"], p["patch"]
    else:
        d.kind, d.n_layers, d.d, d.n_heads = MODEL_DECODER, p["n_layers"], p["d"], p["n_q_heads"]
        d.n_kv_heads, d.head_dim, d.ffn, d.vocab = p["n_kv_heads"], p["head_dim"], p["ffn"], p["vocab"]
        d.kv_pool, d.kv_pages, d.max_kv_len = kv_pool.data_ptr(), kv_pages or kv_pool.shape[1], max_kv_len
        keep.append(kv_pool)
        if trace is not None:
            assert trace.is_cuda and trace.dtype.itemsize == 4 and trace.numel() >= (p["n_layers"] + 1) * max(max_batch, 1) * p["d"]
            d.trace = trace.data_ptr()
            keep.append(trace)
    return d, keep


# ----------------------------------------------------------------------------- context
class Context:
    """Thin owner of an epara_ctx.  Methods mirror the C entry points one to one."""

    def __init__(self, workspace, device: int = 0, cap_ls: int = 0, cap_fs: int = 0, mf_max: int = 0,
                 gemm_impl: int = GEMM_TCGEN05, max_queue: int = 0, profile: bool = False):
        self.cfg = Config(device, workspace.data_ptr(), workspace.numel() * workspace.element_size(), cap_ls, cap_fs,
                          mf_max, gemm_impl, max_queue, int(profile))
        self._keep = [workspace]
        self.h = C.c_void_p()
        _check(lib.epara_init(C.byref(self.cfg), C.byref(self.h)), "epara_init")

    def model_workspace_bytes(self, desc: ModelDesc) -> int:
        return lib.epara_model_workspace_bytes(C.byref(self.cfg), C.byref(desc))

    def epara_register_model(self, desc: ModelDesc, keep=None) -> int:
        mid = C.c_int(-1)
        _check(lib.epara_register_model(self.h, C.byref(desc), C.byref(mid)), "epara_register_model")
        self._keep.append(keep)
        return mid.value

    def epara_submit(self, model_id: int, category: int, inp: Inputs, raise_on_error: bool = True):
        t = C.c_uint64(0)
        s = lib.epara_submit(self.h, model_id, category, C.byref(inp), C.byref(t))
        if raise_on_error:
            _check(s, "epara_submit")
            return t.value
        return s, t.value

    def epara_submit_many(self, model_id: int, category: int, inputs, n: int, tickets=None):
        """inputs: a ctypes array of Inputs; returns the ctypes array of tickets."""
        tk = tickets if tickets is not None else (C.c_uint64 * max(n, 1))()
        acc = C.c_int(0)
        _check(lib.epara_submit_many(self.h, model_id, category, inputs, n, tk, C.byref(acc)), "epara_submit_many")
        return tk

    def epara_step(self, stream_ptr: int, now_ns: int = -1) -> StepInfo:
        info = StepInfo()
        _check(lib.epara_step(self.h, C.c_void_p(stream_ptr), now_ns, C.byref(info)), "epara_step")
        return info

    def epara_collect(self, ticket: int):
        out = Output()
        s = lib.epara_collect(self.h, ticket, C.byref(out))
        return s, out

    def epara_set_profile(self, on: bool):
        _check(lib.epara_set_profile(self.h, int(on)), "epara_set_profile")

    def epara_step_profile(self):
        ms = (C.c_float * K_COUNT)()
        n = (C.c_int * K_COUNT)()
        _check(lib.epara_step_profile(self.h, ms, n), "epara_step_profile")
        return {K_NAMES[i]: (ms[i], n[i]) for i in range(K_COUNT)}

    def close(self):
        if self.h:
            lib.epara_destroy(self.h)
            self.h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ----------------------------------------------------------------------------- single kernels
def gemm_problem_array(problems: Sequence[Dict]):
    n = len(problems)
    arr = (GemmProblem * max(n, 1))()
    for i, p in enumerate(problems):
        arr[i] = GemmProblem(p["A"].data_ptr(), p["W"].data_ptr(), p["C"].data_ptr(),
                             p["bias"].data_ptr() if p.get("bias") is not None else None,
                             p["M"], p["N"], p["K"], p["A"].stride(0), p["W"].stride(0), p["C"].stride(0),
                             p.get("epilogue", 0))
    return arr


def epara_gemm_scratch_bytes_for(problems: Sequence[Dict], device: int = 0) -> int:
    return lib.epara_gemm_scratch_bytes_for(device, gemm_problem_array(problems), len(problems))


def epara_grouped_gemm(problems: Sequence[Dict], stream_ptr: int, scratch, impl: int = GEMM_TCGEN05, device: int = 0):
    """problems: dicts with torch tensors A [M, lda], W [N, ldw], C, optional bias, and M, N, K, epilogue."""
    n = len(problems)
    arr = gemm_problem_array(problems)
    _check(lib.epara_grouped_gemm(device, C.c_void_p(stream_ptr), impl, arr, n, scratch.data_ptr(),
                                  scratch.numel() * scratch.element_size()), "epara_grouped_gemm")


def epara_decode_attention(q, kv_layer, kv_lens, tables, out, Hq: int, Hkv: int, hd: int, max_len: int, scratch,
                           stream_ptr: int, device: int = 0, kv_pages: int = 0):
    """kv_pages: pages of kv_layer the call may touch (default: all of the tensor's)."""
    B = q.shape[0]
    _check(lib.epara_decode_attention(device, C.c_void_p(stream_ptr), q.data_ptr(), q.stride(0), kv_layer.data_ptr(),
                                      kv_pages or kv_layer.shape[0], kv_lens.data_ptr(), tables.data_ptr(), tables.stride(0), out.data_ptr(), B, Hq,
                                      Hkv, hd, max_len, scratch.data_ptr(),
                                      scratch.numel() * scratch.element_size()), "epara_decode_attention")


def epara_decode_attention_static(q, kv_layer, kv_lens, tables, out, Hq: int, Hkv: int, hd: int, max_len: int,
                                  stream_ptr: int, device: int = 0, kv_pages: int = 0):
    """Decode attention for callers that must not allocate: same arguments as epara_decode_attention
    without the scratch tensor (the library's built-in per-GPU array is used instead)."""
    B = q.shape[0]
    _check(lib.epara_decode_attention_static(device, C.c_void_p(stream_ptr), q.data_ptr(), q.stride(0),
                                             kv_layer.data_ptr(), kv_pages or kv_layer.shape[0], kv_lens.data_ptr(),
                                             tables.data_ptr(), tables.stride(0), out.data_ptr(), B, Hq, Hkv, hd,
                                             max_len),
           "epara_decode_attention_static")


def epara_decode_attention_static_status(device: int = 0):
    """(status, code) of the last allocation-free decode-attention call on the device."""
    code = C.c_int(0)
    return lib.epara_decode_attention_static_status(device, C.byref(code)), code.value


def epara_selftest_bounded_wait(status_dev, stream_ptr: int, limit_ns: int = 1_000_000, device: int = 0):
    """(status, code): runs a wait that cannot complete for at most limit_ns; E_DEVICE / 90 is the expected answer."""
    code = C.c_int(0)
    s = lib.epara_selftest_bounded_wait(device, C.c_void_p(stream_ptr), limit_ns, status_dev.data_ptr(), C.byref(code))
    return s, code.value


# ----------------------------------------------------------------------------- host policies (marshalling only)
def _policy_args(cluster: Dict, services: Sequence[Dict], requests: Sequence[Dict]):
    gp = (C.c_int * len(cluster["gpus"]))(*cluster["gpus"])
    cl = Cluster(len(cluster["gpus"]), C.cast(gp, C.POINTER(C.c_int)), cluster["vram"], cluster["sync_ms"], cluster["offload_ms"])
    sv = (Service * max(len(services), 1))()
    for i, s in enumerate(services):
        sv[i] = Service(s["a"], s["b"], s["n_gpus"], s["cat"], s["bs"], s["slo_ms"], s.get("fps", 0.0), s.get("frames", 0),
                        (C.c_double * PROFILE_POINTS)(*s["c_ms"]))
    rq = (SimRequest * max(len(requests), 1))()
    for i, r in enumerate(requests):
        rq[i] = SimRequest(r["t_ms"], r["service"], r["server"], (C.c_double * MAX_OFFLOAD_DRAWS)(*r["u"]))
    return cl, sv, rq, gp


def _placements(pl):
    arr = (Placement * max(len(pl), 1))()
    for i, (l, n) in enumerate(pl):
        arr[i] = Placement(l, n)
    return arr


def epara_offload_probabilities(p_hat, p_act, queued_ms, t_sync_ms, slo_ms: float):
    n = len(p_hat)
    D = C.c_double * max(n, 1)
    out = D()
    _check(lib.epara_offload_probabilities(n, D(*p_hat), D(*p_act), D(*queued_ms), D(*t_sync_ms), slo_ms, out),
           "epara_offload_probabilities")
    return list(out[:n])


def epara_simulate(cluster: Dict, services, requests, placements, max_offload: int = MAX_OFFLOAD_DRAWS) -> Dict:
    cl, sv, rq, _keep = _policy_args(cluster, services, requests)
    res = SimResult()
    _check(lib.epara_simulate(C.byref(cl), sv, len(services), rq, len(requests), _placements(placements), len(placements),
                              max_offload, C.byref(res)), "epara_simulate")
    return {k: getattr(res, k) for k, _ in SimResult._fields_}


def epara_place_sssp(cluster: Dict, services, requests, priority, max_offload: int = MAX_OFFLOAD_DRAWS, cap: int = 4096):
    cl, sv, rq, _keep = _policy_args(cluster, services, requests)
    out = (Placement * cap)()
    n = C.c_int(0)
    _check(lib.epara_place_sssp(C.byref(cl), sv, len(services), rq, len(requests), _placements(priority), len(priority),
                                max_offload, out, cap, C.byref(n)), "epara_place_sssp")
    return [(out[i].service, out[i].server) for i in range(n.value)]
