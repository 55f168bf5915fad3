"""Thin Python binding of the C-ABI library (libqzo.so): argument marshalling only.

Every function has the name of the C entry point it calls and takes torch CUDA tensors
where the C function takes device pointers.  PyTorch is used for device memory and
streams; every step of the path runs in the library's kernels.  There is no fallback:
if the shared library is missing or fails to load, importing this module raises.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqzo.so")

QZO_OK = 0
ERR_BAD_ARG, ERR_UNSUPPORTED_DEVICE, ERR_WORKSPACE, ERR_NONFINITE = -1, -2, -3, -4
ERR_DEVICE_TIMEOUT, ERR_CUDA, ERR_MISSING_TENSOR = -5, -6, -7
ARCH = {"llama": 0, "opt": 1}
DTYPE = {torch.bfloat16: 0, torch.float32: 1, torch.int32: 3}
DTYPE_U32 = 2

EXPORTS = (
    "qzo_strerror", "qzo_last_cuda_error", "qzo_philox_words", "qzo_normals", "qzo_quantize_int4",
    "qzo_unpack_int4", "qzo_repacked_bytes", "qzo_repack_int4", "qzo_unpack_kernel_layout",
    "qzo_gemm_workspace_bytes", "qzo_perturbed_gemm", "qzo_perturbed_gemm_noalloc", "qzo_update_scales_flat", "qzo_num_scales",
    "qzo_scale_layout", "qzo_workspace_bytes", "qzo_init_model", "qzo_free_model", "qzo_forward_loss",
    "qzo_update_scales", "qzo_step", "qzo_step_host", "qzo_debug_set_capture", "qzo_debug_layer_output",
    "qzo_device_status", "qzo_launch_count", "qzo_profile_gemms", "qzo_profile_read",
    "qzo_step_begin", "qzo_step_finish", "qzo_get_scales", "qzo_set_scales", "qzo_debug_set_status", "qzo_use_recorded_steps", "qzo_recorded_step_count", "qzo_perturbed_gemm_codebook16_channelwise",
    "qzo_joint_workspace_bytes", "qzo_enable_joint_spsa", "qzo_perturbed_gemm_table16", "qzo_debug_gemm_wait_expiry",
)


class QzoError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        msg = _lib.qzo_strerror(status).decode()
        if status == ERR_CUDA:
            msg += f" [cudaError {_lib.qzo_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} ({status})")


class ModelDesc(ctypes.Structure):
    _fields_ = [("arch", ctypes.c_int), ("n_layers", ctypes.c_int), ("d_model", ctypes.c_int),
                ("n_heads", ctypes.c_int), ("d_ffn", ctypes.c_int), ("vocab", ctypes.c_int),
                ("max_seq", ctypes.c_int), ("group_size", ctypes.c_int),
                ("norm_eps", ctypes.c_float), ("rope_theta", ctypes.c_float)]


class Tensor(ctypes.Structure):
    _fields_ = [("name", ctypes.c_char_p), ("dptr", ctypes.c_void_p), ("dtype", ctypes.c_int),
                ("shape", ctypes.c_int64 * 2)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with paper_2505_13430_b200/build.py "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, u64, i64, ci, cf, sz = (ctypes.c_void_p, ctypes.c_uint64, ctypes.c_int64, ctypes.c_int,
                                ctypes.c_float, ctypes.c_size_t)
    P = ctypes.POINTER
    sig = {
        "qzo_strerror": (ctypes.c_char_p, [ci]),
        "qzo_last_cuda_error": (ci, []),
        "qzo_launch_count": (i64, []),
        "qzo_philox_words": (ci, [u64, u64, i64, vp, vp, vp]),
        "qzo_normals": (ci, [u64, u64, i64, vp, vp]),
        "qzo_quantize_int4": (ci, [vp, ci, ci, vp, vp, vp]),
        "qzo_unpack_int4": (ci, [vp, ci, ci, vp, vp]),
        "qzo_repacked_bytes": (ci, [ci, ci, P(sz)]),
        "qzo_repack_int4": (ci, [vp, ci, ci, vp, sz, vp]),
        "qzo_unpack_kernel_layout": (ci, [vp, ci, ci, vp, vp]),
        "qzo_gemm_workspace_bytes": (ci, [ci, ci, ci, P(sz)]),
        "qzo_perturbed_gemm": (ci, [vp, vp, vp, vp, vp, ci, ci, ci, u64, u64, ci, cf, vp, sz, vp, vp]),
        "qzo_perturbed_gemm_table16": (ci, [vp, vp, vp, P(cf), vp, vp, ci, ci, ci, u64, u64, ci, cf, vp, sz, vp, vp]),
        "qzo_perturbed_gemm_codebook16_channelwise": (ci, [vp, vp, vp, P(cf), vp, vp, ci, ci, ci, u64, u64, ci, cf, vp, sz, vp, vp]),
        "qzo_debug_gemm_wait_expiry": (ci, [vp, vp, vp, vp, ci, ci, ci, ci, i64, vp, vp]),
        "qzo_perturbed_gemm_noalloc": (ci, [vp, vp, vp, vp, vp, ci, ci, ci, u64, u64, ci, cf, vp, vp]),
        "qzo_update_scales_flat": (ci, [vp, i64, u64, u64, cf, cf, cf, vp]),
        "qzo_num_scales": (ci, [P(ModelDesc), P(i64), P(i64)]),
        "qzo_scale_layout": (ci, [P(ModelDesc), ci, ci, P(i64), P(ci), P(ci)]),
        "qzo_workspace_bytes": (ci, [P(ModelDesc), ci, P(sz)]),
        "qzo_init_model": (ci, [P(ModelDesc), P(Tensor), ci, vp, sz, ci, vp, P(vp)]),
        "qzo_free_model": (ci, [vp]),
        "qzo_forward_loss": (ci, [vp, vp, vp, ci, ci, u64, ci, cf, vp]),
        "qzo_update_scales": (ci, [vp, u64, cf, cf, cf]),
        "qzo_step": (ci, [vp, vp, vp, ci, ci, u64, cf, cf, cf, vp]),
        "qzo_step_host": (ci, [vp, vp, vp, ci, ci, u64, cf, cf, cf, vp]),
        "qzo_step_begin": (ci, [vp, vp, vp, ci, ci, u64, cf, vp]),
        "qzo_step_finish": (ci, [vp, vp, u64, cf, cf, cf, vp]),
        "qzo_get_scales": (ci, [vp, ci, vp, sz]),
        "qzo_set_scales": (ci, [vp, ci, vp, sz]),
        "qzo_debug_set_status": (ci, [vp, ci]),
        "qzo_use_recorded_steps": (ci, [vp, ci]),
        "qzo_recorded_step_count": (ci, [vp, vp]),
        "qzo_joint_workspace_bytes": (ci, [P(ModelDesc), P(sz)]),
        "qzo_enable_joint_spsa": (ci, [vp, vp, sz, cf]),
        "qzo_debug_set_capture": (ci, [vp, ci]),
        "qzo_debug_layer_output": (ci, [vp, ci, ci, vp, sz]),
        "qzo_device_status": (ci, [vp, P(ci)]),
        "qzo_profile_gemms": (ci, [vp, ci]),
        "qzo_profile_read": (ci, [vp, P(i64), P(ctypes.c_double), P(ctypes.c_double)]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


_lib = _load()


def _check(status, where):
    if status != QZO_OK:
        raise QzoError(status, where)


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else ctypes.c_void_p(0)


def _cuda(t, dtype=None):
    assert t.is_cuda and t.is_contiguous(), "expects a contiguous CUDA tensor"
    if dtype is not None:
        assert t.dtype == dtype, f"expects {dtype}, got {t.dtype}"
    return t


def qzo_launch_count():
    return int(_lib.qzo_launch_count())


def qzo_philox_words(seed, block_base, n_blocks, with_uniforms=True):
    """-> (int32 [n_blocks][4] holding the uint32 words, float32 [n_blocks][4] uniforms or None)."""
    words = torch.empty((n_blocks, 4), dtype=torch.int32, device="cuda")
    uni = torch.empty((n_blocks, 4), dtype=torch.float32, device="cuda") if with_uniforms else None
    _check(_lib.qzo_philox_words(seed, block_base, n_blocks, _ptr(words), _ptr(uni), _stream()), "qzo_philox_words")
    return words, uni


def qzo_normals(seed, index_base, count):
    z = torch.empty((count,), dtype=torch.float32, device="cuda")
    _check(_lib.qzo_normals(seed, index_base, count, _ptr(z), _stream()), "qzo_normals")
    return z


def qzo_quantize_int4(w):
    """float32 [K][N] -> (int32 [K/8][N] interchange words, bf16 [G][N] scales)."""
    _cuda(w, torch.float32)
    K, N = w.shape
    packed = torch.empty((K // 8, N), dtype=torch.int32, device=w.device)
    scales = torch.empty(((K + 127) // 128, N), dtype=torch.bfloat16, device=w.device)
    _check(_lib.qzo_quantize_int4(_ptr(w), K, N, _ptr(packed), _ptr(scales), _stream()), "qzo_quantize_int4")
    return packed, scales


def qzo_unpack_int4(packed, K, N):
    _cuda(packed, torch.int32)
    q = torch.empty((K, N), dtype=torch.int8, device=packed.device)
    _check(_lib.qzo_unpack_int4(_ptr(packed), K, N, _ptr(q), _stream()), "qzo_unpack_int4")
    return q


def qzo_repacked_bytes(K, N):
    out = ctypes.c_size_t(0)
    _check(_lib.qzo_repacked_bytes(K, N, ctypes.byref(out)), "qzo_repacked_bytes")
    return out.value


def qzo_repack_int4(packed, K, N):
    """interchange words -> kernel-layout bytes (uint8 tensor)."""
    _cuda(packed, torch.int32)
    nbytes = qzo_repacked_bytes(K, N)
    out = torch.empty((nbytes,), dtype=torch.uint8, device=packed.device)
    _check(_lib.qzo_repack_int4(_ptr(packed), K, N, _ptr(out), nbytes, _stream()), "qzo_repack_int4")
    return out


def qzo_unpack_kernel_layout(wq, K, N):
    _cuda(wq, torch.uint8)
    q = torch.empty((K, N), dtype=torch.int8, device=wq.device)
    _check(_lib.qzo_unpack_kernel_layout(_ptr(wq), K, N, _ptr(q), _stream()), "qzo_unpack_kernel_layout")
    return q


def qzo_gemm_workspace_bytes(M, K, N):
    out = ctypes.c_size_t(0)
    _check(_lib.qzo_gemm_workspace_bytes(M, K, N, ctypes.byref(out)), "qzo_gemm_workspace_bytes")
    return out.value


def qzo_perturbed_gemm(x, wq, scales, M, K, N, seed, scale_index_base, sign, eps, bias=None, y=None,
                       workspace=None, status=None):
    """Y = X W' with W' de-quantised from int4 and s' = s + sign*eps*z.  Returns bf16 [M][N]."""
    _cuda(x, torch.bfloat16), _cuda(wq, torch.uint8), _cuda(scales, torch.bfloat16)
    if y is None:
        y = torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
    need = qzo_gemm_workspace_bytes(M, K, N)
    if workspace is None and need:
        workspace = torch.empty((need,), dtype=torch.uint8, device=x.device)
    ws_bytes = workspace.numel() if workspace is not None else 0
    _check(_lib.qzo_perturbed_gemm(_ptr(x), _ptr(wq), _ptr(scales), _ptr(bias), _ptr(y), M, K, N, seed,
                                   scale_index_base, sign, eps, _ptr(workspace), ws_bytes, _ptr(status), _stream()),
           "qzo_perturbed_gemm")
    return y


def qzo_perturbed_gemm_table16(x, codes_wq, scales, table16, M, K, N, seed, scale_index_base, sign, eps, bias=None, y=None,
                               workspace=None, status=None):
    """Y = X W' for 4-bit codes into a 16-entry table with one bf16 scale per block of 64 rows (NF4-style storage);
    codes_wq is qzo_repack_int4 of the codes packed like int4 nibbles; table16: 16 floats (any sequence)."""
    _cuda(x, torch.bfloat16), _cuda(codes_wq, torch.uint8), _cuda(scales, torch.bfloat16)
    assert scales.shape[0] == (K + 63) // 64
    if y is None:
        y = torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
    need = qzo_gemm_workspace_bytes(M, K, N)
    if workspace is None and need:
        workspace = torch.empty((need,), dtype=torch.uint8, device=x.device)
    ws_bytes = workspace.numel() if workspace is not None else 0
    table = (ctypes.c_float * 16)(*[float(v) for v in table16])
    _check(_lib.qzo_perturbed_gemm_table16(_ptr(x), _ptr(codes_wq), _ptr(scales), table, _ptr(bias), _ptr(y), M, K, N, seed,
                                           scale_index_base, sign, eps, _ptr(workspace), ws_bytes, _ptr(status), _stream()),
           "qzo_perturbed_gemm_table16")
    return y


def qzo_perturbed_gemm_codebook16_channelwise(x, codes_wq, scales, table16, M, K, N, seed, scale_index_base, sign, eps,
                                              bias=None, y=None, workspace=None, status=None):
    """Y = X W' for 4-bit codes into a 16-entry table with ONE bf16 scale per output channel (scales: [N]);
    codes_wq as for qzo_perturbed_gemm_table16."""
    _cuda(x, torch.bfloat16), _cuda(codes_wq, torch.uint8), _cuda(scales, torch.bfloat16)
    assert scales.numel() == N
    if y is None:
        y = torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
    need = qzo_gemm_workspace_bytes(M, K, N)
    if workspace is None and need:
        workspace = torch.empty((need,), dtype=torch.uint8, device=x.device)
    ws_bytes = workspace.numel() if workspace is not None else 0
    table = (ctypes.c_float * 16)(*[float(v) for v in table16])
    _check(_lib.qzo_perturbed_gemm_codebook16_channelwise(_ptr(x), _ptr(codes_wq), _ptr(scales), table, _ptr(bias), _ptr(y),
                                                          M, K, N, seed, scale_index_base, sign, eps, _ptr(workspace),
                                                          ws_bytes, _ptr(status), _stream()),
           "qzo_perturbed_gemm_codebook16_channelwise")
    return y


def qzo_debug_gemm_wait_expiry(x, wq, scales, y, M, K, N, skip_group, wait_limit_cycles, status):
    """Test entry: the GEMM with one group's copies withheld and a short wait limit; see include/qzo.h."""
    _cuda(x, torch.bfloat16), _cuda(wq, torch.uint8), _cuda(scales, torch.bfloat16), _cuda(y, torch.bfloat16)
    _check(_lib.qzo_debug_gemm_wait_expiry(_ptr(x), _ptr(wq), _ptr(scales), _ptr(y), M, K, N, skip_group, wait_limit_cycles,
                                           _ptr(status), _stream()), "qzo_debug_gemm_wait_expiry")


NOALLOC_SCRATCH_BYTES = 16 << 20


def qzo_perturbed_gemm_noalloc(x, wq, scales, y, M, K, N, seed, scale_index_base, sign, eps, bias=None, status=None):
    """qzo_perturbed_gemm for callers that cannot allocate: no workspace argument (the library's
    fixed scratch array is used) and the output tensor y is the caller's.  Nothing is allocated here."""
    _cuda(x, torch.bfloat16), _cuda(wq, torch.uint8), _cuda(scales, torch.bfloat16), _cuda(y, torch.bfloat16)
    _check(_lib.qzo_perturbed_gemm_noalloc(_ptr(x), _ptr(wq), _ptr(scales), _ptr(bias), _ptr(y), M, K, N, seed,
                                           scale_index_base, sign, eps, _ptr(status), _stream()),
           "qzo_perturbed_gemm_noalloc")
    return y


def qzo_update_scales_flat(scales, seed, index_base, lr, g, clip):
    _cuda(scales, torch.bfloat16)
    _check(_lib.qzo_update_scales_flat(_ptr(scales), scales.numel(), seed, index_base, lr, g, clip, _stream()),
           "qzo_update_scales_flat")
    return scales


def make_desc(cfg):
    return ModelDesc(ARCH[cfg["arch"]], cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["d_ffn"],
                     cfg["vocab"], cfg["max_seq"], 128, cfg["norm_eps"], cfg["rope_theta"])


def qzo_num_scales(cfg):
    flat, train = ctypes.c_int64(0), ctypes.c_int64(0)
    d = make_desc(cfg)
    _check(_lib.qzo_num_scales(ctypes.byref(d), ctypes.byref(flat), ctypes.byref(train)), "qzo_num_scales")
    return flat.value, train.value


def qzo_scale_layout(cfg, layer, linear):
    base, G, N = ctypes.c_int64(0), ctypes.c_int(0), ctypes.c_int(0)
    d = make_desc(cfg)
    _check(_lib.qzo_scale_layout(ctypes.byref(d), layer, linear, ctypes.byref(base), ctypes.byref(G),
                                 ctypes.byref(N)), "qzo_scale_layout")
    return base.value, G.value, N.value


def qzo_workspace_bytes(cfg, max_tokens):
    out = ctypes.c_size_t(0)
    d = make_desc(cfg)
    _check(_lib.qzo_workspace_bytes(ctypes.byref(d), max_tokens, ctypes.byref(out)), "qzo_workspace_bytes")
    return out.value


class Model:
    """Owns the device tensors of a model (allocated by torch) and the library handle.

    tensors: dict name -> CUDA tensor with the names qzo_init_model documents; "*.qweight"
    tensors are int32 holding the interchange words and may be dropped after construction.
    """

    def __init__(self, cfg, tensors, max_tokens):
        self.cfg = dict(cfg)
        self.max_tokens = max_tokens
        self.desc = make_desc(cfg)
        self.scales = tensors["scales"]
        self._keep = {k: v for k, v in tensors.items() if not k.endswith(".qweight")}
        nbytes = qzo_workspace_bytes(cfg, max_tokens)
        self.workspace = torch.empty((nbytes,), dtype=torch.uint8, device="cuda")
        arr = (Tensor * len(tensors))()
        for i, (name, t) in enumerate(tensors.items()):
            _cuda(t)
            dt = DTYPE_U32 if name.endswith(".qweight") else DTYPE[t.dtype]
            shape = (t.shape[0], t.shape[1] if t.dim() > 1 else 1)
            arr[i] = Tensor(name.encode(), t.data_ptr(), dt, (ctypes.c_int64 * 2)(*shape))
        handle = ctypes.c_void_p(0)
        self.stream = torch.cuda.current_stream()
        _check(_lib.qzo_init_model(ctypes.byref(self.desc), arr, len(tensors), _ptr(self.workspace), nbytes,
                                   max_tokens, ctypes.c_void_p(self.stream.cuda_stream), ctypes.byref(handle)),
               "qzo_init_model")
        self.handle = handle
        self.stream.synchronize()
        self._loss = torch.zeros((2,), dtype=torch.float32, device="cuda")

    def close(self):
        if self.handle:
            _lib.qzo_free_model(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def qzo_forward_loss(self, tokens, labels, seed, sign, eps, loss_out=None):
        _cuda(tokens, torch.int32), _cuda(labels, torch.int32)
        B, S = tokens.shape
        out = self._loss[:1] if loss_out is None else loss_out
        _check(_lib.qzo_forward_loss(self.handle, _ptr(tokens), _ptr(labels), B, S, seed, sign, eps, _ptr(out)),
               "qzo_forward_loss")
        return out

    def qzo_update_scales(self, seed, lr, g, clip):
        _check(_lib.qzo_update_scales(self.handle, seed, lr, g, clip), "qzo_update_scales")

    def qzo_step(self, tokens, labels, seed, eps, lr, clip, read_back=True):
        _cuda(tokens, torch.int32), _cuda(labels, torch.int32)
        B, S = tokens.shape
        out = (ctypes.c_float * 4)() if read_back else None
        _check(_lib.qzo_step(self.handle, _ptr(tokens), _ptr(labels), B, S, seed, eps, lr, clip, out), "qzo_step")
        return tuple(out) if read_back else None

    def qzo_step_begin(self, tokens, labels, seed, eps, sums=None):
        """-> float32 CUDA tensor [4]: sum of token losses (+), the same (-), kept tokens (+), (-)."""
        _cuda(tokens, torch.int32), _cuda(labels, torch.int32)
        B, S = tokens.shape
        if sums is None:
            sums = torch.empty((4,), dtype=torch.float32, device="cuda")
        _check(_lib.qzo_step_begin(self.handle, _ptr(tokens), _ptr(labels), B, S, seed, eps, _ptr(sums)),
               "qzo_step_begin")
        return sums

    def qzo_step_finish(self, sums, seed, eps, lr, clip, read_back=True):
        _cuda(sums, torch.float32)
        out = (ctypes.c_float * 4)() if read_back else None
        _check(_lib.qzo_step_finish(self.handle, _ptr(sums), seed, eps, lr, clip, out), "qzo_step_finish")
        return tuple(out) if read_back else None

    def _linear_bytes(self, linear_id):
        if linear_id == -1:
            return self.scales.numel() * 2
        n_lin = 7 if self.cfg["arch"] == "llama" else 6
        _, G, N = qzo_scale_layout(self.cfg, linear_id // n_lin, linear_id % n_lin)
        return G * N * 2

    def qzo_get_scales(self, linear_id, out=None):
        """Copy of one linear's scales (bf16, flat [G*N]) or of the whole flat buffer (linear_id = -1)."""
        if out is None:
            out = torch.empty((self._linear_bytes(linear_id) // 2,), dtype=torch.bfloat16, device="cuda")
        _check(_lib.qzo_get_scales(self.handle, linear_id, _ptr(out), out.numel() * 2), "qzo_get_scales")
        return out

    def qzo_set_scales(self, linear_id, values):
        _cuda(values, torch.bfloat16)
        _check(_lib.qzo_set_scales(self.handle, linear_id, _ptr(values), values.numel() * 2), "qzo_set_scales")

    def qzo_enable_joint_spsa(self, lr_dense, on=True):
        """Joint mode: embed, lm_head and the norm vectors are perturbed and updated too (plain SPSA)."""
        if not on:
            _check(_lib.qzo_enable_joint_spsa(self.handle, None, 0, 0.0), "qzo_enable_joint_spsa")
            return
        need = ctypes.c_size_t(0)
        _check(_lib.qzo_joint_workspace_bytes(ctypes.byref(self.desc), ctypes.byref(need)), "qzo_joint_workspace_bytes")
        self._joint_ws = torch.empty((need.value,), dtype=torch.uint8, device="cuda")
        _check(_lib.qzo_enable_joint_spsa(self.handle, _ptr(self._joint_ws), need.value, lr_dense), "qzo_enable_joint_spsa")

    def tensor(self, name):
        """The caller-owned device tensor bound under `name` at construction (e.g. "embed", "L0.norm1_w")."""
        return self._keep[name]

    def qzo_debug_set_status(self, value):
        _check(_lib.qzo_debug_set_status(self.handle, value), "qzo_debug_set_status")

    def qzo_use_recorded_steps(self, on):
        _check(_lib.qzo_use_recorded_steps(self.handle, 1 if on else 0), "qzo_use_recorded_steps")

    def qzo_recorded_step_count(self):
        n = ctypes.c_int(0)
        _check(_lib.qzo_recorded_step_count(self.handle, ctypes.byref(n)), "qzo_recorded_step_count")
        return n.value

    def qzo_step_host(self, tokens_host, labels_host, seed, eps, lr, clip):
        assert not tokens_host.is_cuda and tokens_host.dtype == torch.int32 and tokens_host.is_contiguous()
        B, S = tokens_host.shape
        out = (ctypes.c_float * 4)()
        _check(_lib.qzo_step_host(self.handle, ctypes.c_void_p(tokens_host.data_ptr()),
                                  ctypes.c_void_p(labels_host.data_ptr()), B, S, seed, eps, lr, clip, out),
               "qzo_step_host")
        return tuple(out)

    def qzo_debug_set_capture(self, layer):
        _check(_lib.qzo_debug_set_capture(self.handle, layer), "qzo_debug_set_capture")

    def qzo_debug_layer_output(self, layer, which, T):
        if which == 0:
            out = torch.empty((T, self.cfg["d_model"]), dtype=torch.bfloat16, device="cuda")
        else:
            out = torch.empty((T, self.cfg["vocab"]), dtype=torch.float32, device="cuda")
        _check(_lib.qzo_debug_layer_output(self.handle, layer, which, _ptr(out), out.numel() * out.element_size()),
               "qzo_debug_layer_output")
        return out

    def qzo_device_status(self):
        st = ctypes.c_int(0)
        rc = _lib.qzo_device_status(self.handle, ctypes.byref(st))
        if rc not in (QZO_OK, ERR_DEVICE_TIMEOUT, ERR_BAD_ARG):
            _check(rc, "qzo_device_status")
        return st.value

    def qzo_profile_gemms(self, max_launches):
        _check(_lib.qzo_profile_gemms(self.handle, max_launches), "qzo_profile_gemms")

    def qzo_profile_read(self):
        """-> (launches, total_ms, total_flops) of the bracketed GEMM launches since the last read."""
        n, ms, fl = ctypes.c_int64(0), ctypes.c_double(0), ctypes.c_double(0)
        _check(_lib.qzo_profile_read(self.handle, ctypes.byref(n), ctypes.byref(ms), ctypes.byref(fl)),
               "qzo_profile_read")
        return n.value, ms.value, fl.value

    def scales_of(self, layer, linear):
        """View of one linear's scales [G][N] inside the flat buffer."""
        base, G, N = qzo_scale_layout(self.cfg, layer, linear)
        return self.scales[base:base + G * N].view(G, N)


def build_model_from_raw(raw, max_tokens, quantized=None):
    """Quantise (library kernel) and upload the seeded raw tensors of `inputs.raw_model_tensors`.

    quantized: optional dict (layer, name) -> (int32 words [K/8][N], bf16 scales [G][N]) to use instead
    of quantising here.  Returns Model.
    """
    from .inputs import linear_shapes
    cfg = raw["cfg"]
    flat, _ = qzo_num_scales(cfg)
    scales = torch.zeros((flat,), dtype=torch.bfloat16, device="cuda")
    t = {"embed": raw["embed"].cuda(), "lm_head": raw["lm_head"].cuda(),
         "final_norm_w": raw["final_norm_w"].float().cuda(), "scales": scales}
    if cfg["arch"] == "opt":
        t["pos_embed"] = raw["pos_embed"].cuda()
        t["final_norm_b"] = raw["final_norm_b"].float().cuda()
    for li, layer in enumerate(raw["layers"]):
        for k in ("norm1_w", "norm2_w", "norm1_b", "norm2_b"):
            if k in layer:
                t[f"L{li}.{k}"] = layer[k].float().cuda()
        for idx, (name, K, N) in enumerate(linear_shapes(cfg)):
            ent = layer["lin"][name]
            if quantized is not None:
                words, s = quantized[(li, name)]
                words, s = words.cuda(), s.cuda()
            else:
                words, s = qzo_quantize_int4(ent["w"].cuda().contiguous())
            base, G, Nn = qzo_scale_layout(cfg, li, idx)
            scales[base:base + G * Nn] = s.reshape(-1)
            t[f"L{li}.{name}.qweight"] = words
            if "bias" in ent:
                t[f"L{li}.{name}.bias"] = ent["bias"].float().cuda()
    return Model(cfg, t, max_tokens)


def build_random_model_gpu(cfg, max_tokens, seed=1000):
    """Random-init int4 model generated and quantised tensor by tensor on the device
    (fp32 N(0, 0.02) weights -> library quantiser), so that no full-precision copy of the
    model ever exists.  Used by the benchmark for the large configurations."""
    from .inputs import linear_shapes, normal_fp32
    flat, _ = qzo_num_scales(cfg)
    d, V = cfg["d_model"], cfg["vocab"]
    sid = [int(seed)]

    def nxt():
        sid[0] += 1
        return sid[0]

    scales = torch.zeros((flat,), dtype=torch.bfloat16, device="cuda")
    t = {"embed": normal_fp32((V, d), 0.02, nxt(), "cuda").bfloat16(),
         "lm_head": normal_fp32((V, d), 0.02, nxt(), "cuda").bfloat16(),
         "final_norm_w": torch.ones(d, device="cuda"), "scales": scales}
    opt = cfg["arch"] == "opt"
    if opt:
        t["pos_embed"] = normal_fp32((cfg["max_seq"], d), 0.02, nxt(), "cuda").bfloat16()
        t["final_norm_b"] = torch.zeros(d, device="cuda")
    for li in range(cfg["n_layers"]):
        t[f"L{li}.norm1_w"] = torch.ones(d, device="cuda")
        t[f"L{li}.norm2_w"] = torch.ones(d, device="cuda")
        if opt:
            t[f"L{li}.norm1_b"] = torch.zeros(d, device="cuda")
            t[f"L{li}.norm2_b"] = torch.zeros(d, device="cuda")
        for idx, (name, K, N) in enumerate(linear_shapes(cfg)):
            w = normal_fp32((K, N), 0.02, nxt(), "cuda")
            words, s = qzo_quantize_int4(w)
            del w
            base, G, Nn = qzo_scale_layout(cfg, li, idx)
            scales[base:base + G * Nn] = s.reshape(-1)
            t[f"L{li}.{name}.qweight"] = words
            if opt:
                t[f"L{li}.{name}.bias"] = normal_fp32((N,), 0.02, nxt(), "cuda")
    m = Model(cfg, t, max_tokens)
    del t
    torch.cuda.empty_cache()
    return m
