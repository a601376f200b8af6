"""ctypes binding of libsantapp.so: argument marshalling only.

Every step of the path (team build, routing, sampling, exact attention, split-K
merge) runs in the library's CUDA kernels. PyTorch is used for device memory and
streams. There is no CPU fallback: if the library is missing or cannot be loaded
the first call raises.

The functions keep the names of the C entry points (include/santapp.h, include/santapp_latent.h).
"""
import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsantapp.so")

SANTAPP_OK = 0
SANTAPP_ERR_INVALID_ARG = -1
SANTAPP_ERR_UNSUPPORTED = -2
SANTAPP_ERR_WORKSPACE_TOO_SMALL = -3
SANTAPP_ERR_CUDA = -4
SANTAPP_ERR_STATIC_SCRATCH = -5
SANTAPP_STATIC_SCRATCH_BYTES = 2 << 20
SANTAPP_BF16, SANTAPP_FP16 = 0, 1

EXPORTS = [
    "santapp_version", "santapp_strerror", "santapp_last_cuda_error", "santapp_build_teams_sizes",
    "santapp_build_teams", "santapp_decode_workspace_bytes", "santapp_decode_attn",
    "santapp_dense_workspace_bytes", "santapp_dense_decode_attn", "santapp_last_launch_count",
    "santapp_set_stage_mask", "santapp_dense_decode_attn_noalloc", "santapp_build_groups_mean",
    "santapp_kmeans_parent_count", "santapp_assign_parents_workspace_bytes", "santapp_assign_parents",
    "santapp_parent_teams_sizes", "santapp_build_teams_parents", "santapp_build_groups_mean_parents",
    "santapp_kmeans_fit_workspace_bytes", "santapp_kmeans_fit",
    "santapp_latent_sizes", "santapp_latent_build_teams", "santapp_latent_decode_workspace_bytes",
    "santapp_latent_decode_attn", "santapp_latent_dense_workspace_bytes", "santapp_latent_dense_decode_attn",
]
LATENT_DIM, LATENT_ROPE_DIM, LATENT_ROW = 512, 64, 576

STAGE_ROUTE, STAGE_SELECT, STAGE_ATTEND, STAGE_MERGE, STAGE_ALL = 1, 2, 4, 8, 15


class SantappError(RuntimeError):
    def __init__(self, status, detail=""):
        self.status = status
        super().__init__(f"santapp status {status}: {detail}")


class CGeom(ctypes.Structure):
    _fields_ = [("n_seqs", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("parent_size", ctypes.c_int32),
                ("reps_per_parent", ctypes.c_int32), ("elem_type", ctypes.c_int32)]


class CSizes(ctypes.Structure):
    _fields_ = [("rows_total", ctypes.c_int64), ("teams_total", ctypes.c_int64),
                ("max_teams_per_seq", ctypes.c_int32), ("max_rows_per_seq", ctypes.c_int32),
                ("team_row_start_elems", ctypes.c_int64), ("build_workspace_bytes", ctypes.c_size_t)]


class CTeams(ctypes.Structure):
    _fields_ = [("k_packed", ctypes.c_void_p), ("v_packed", ctypes.c_void_p), ("rep_keys", ctypes.c_void_p),
                ("team_row_start", ctypes.c_void_p), ("row_token", ctypes.c_void_p),
                ("seq_row_off", ctypes.c_void_p), ("seq_team_off", ctypes.c_void_p),
                ("rep_abs_max", ctypes.c_void_p), ("team_count", ctypes.c_void_p),
                ("rows_total", ctypes.c_int64), ("teams_total", ctypes.c_int64),
                ("max_teams_per_seq", ctypes.c_int32), ("max_rows_per_seq", ctypes.c_int32)]


class CKmeansOpts(ctypes.Structure):
    _fields_ = [("batch_size", ctypes.c_int32), ("max_iter", ctypes.c_int32), ("patience", ctypes.c_int32),
                ("no_host_poll", ctypes.c_int32), ("reassignment_ratio", ctypes.c_double), ("seed", ctypes.c_uint64),
                ("stream_base", ctypes.c_uint32), ("reserved2", ctypes.c_uint32)]


class CDebug(ctypes.Structure):
    _fields_ = [("sel_idx", ctypes.c_void_p), ("sel_logc", ctypes.c_void_p), ("tau", ctypes.c_void_p),
                ("union_rows", ctypes.c_void_p), ("status", ctypes.c_void_p), ("trace", ctypes.c_void_p)]


_lib = None


class CLatentGeom(ctypes.Structure):
    _fields_ = [("n_seqs", ctypes.c_int32), ("n_heads", ctypes.c_int32), ("parent_size", ctypes.c_int32),
                ("reps_per_parent", ctypes.c_int32)]


class CLatentTeams(ctypes.Structure):
    _fields_ = [("rows_packed", ctypes.c_void_p), ("rep_rows", ctypes.c_void_p), ("team_row_start", ctypes.c_void_p),
                ("row_token", ctypes.c_void_p), ("seq_row_off", ctypes.c_void_p), ("seq_team_off", ctypes.c_void_p),
                ("rep_abs_max", ctypes.c_void_p), ("rows_total", ctypes.c_int64), ("teams_total", ctypes.c_int64),
                ("max_teams_per_seq", ctypes.c_int32), ("max_rows_per_seq", ctypes.c_int32)]


def load_library(path: Optional[str] = None):
    """Load libsantapp.so and declare its signatures. Raises if it is missing."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise SantappError(SANTAPP_ERR_CUDA, f"{p} not found: build it with `python -m paper_2609_35629_b200.build` "
                                             "(there is no CPU fallback)")
    L = ctypes.CDLL(p)
    vp, i32, u32, u64, f32, sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint32, ctypes.c_uint64,
                                  ctypes.c_float, ctypes.c_size_t)
    L.santapp_version.restype = ctypes.c_int
    L.santapp_strerror.argtypes = [ctypes.c_int]
    L.santapp_strerror.restype = ctypes.c_char_p
    L.santapp_last_cuda_error.restype = ctypes.c_char_p
    L.santapp_last_launch_count.restype = ctypes.c_int
    L.santapp_build_teams_sizes.argtypes = [ctypes.POINTER(CGeom), ctypes.POINTER(i32), ctypes.POINTER(CSizes)]
    L.santapp_build_teams_sizes.restype = ctypes.c_int
    L.santapp_build_teams.argtypes = [ctypes.POINTER(CGeom), ctypes.POINTER(i32), vp, vp,
                                      ctypes.POINTER(CTeams), vp, sz, vp]
    L.santapp_build_teams.restype = ctypes.c_int
    L.santapp_build_groups_mean.argtypes = L.santapp_build_teams.argtypes
    L.santapp_build_groups_mean.restype = ctypes.c_int
    L.santapp_kmeans_fit_workspace_bytes.argtypes = [ctypes.POINTER(CGeom), ctypes.POINTER(i32), ctypes.POINTER(i32),
                                                     ctypes.POINTER(CKmeansOpts)]
    L.santapp_kmeans_fit_workspace_bytes.restype = sz
    L.santapp_kmeans_fit.argtypes = [ctypes.POINTER(CGeom), ctypes.POINTER(i32), ctypes.POINTER(i32), vp,
                                     ctypes.POINTER(CKmeansOpts), vp, vp, vp, sz, vp]
    L.santapp_kmeans_fit.restype = ctypes.c_int
    L.santapp_kmeans_parent_count.argtypes = [i32, i32]
    L.santapp_kmeans_parent_count.restype = i32
    L.santapp_assign_parents_workspace_bytes.argtypes = [ctypes.POINTER(CGeom)]
    L.santapp_assign_parents_workspace_bytes.restype = sz
    L.santapp_assign_parents.argtypes = [ctypes.POINTER(CGeom), ctypes.POINTER(i32), ctypes.POINTER(i32), vp, vp, vp,
                                         vp, sz, vp]
    L.santapp_assign_parents.restype = ctypes.c_int
    L.santapp_parent_teams_sizes.argtypes = [ctypes.POINTER(CGeom), ctypes.POINTER(i32), ctypes.POINTER(i32),
                                             ctypes.POINTER(CSizes)]
    L.santapp_parent_teams_sizes.restype = ctypes.c_int
    L.santapp_build_teams_parents.argtypes = [ctypes.POINTER(CGeom), ctypes.POINTER(i32), ctypes.POINTER(i32), vp, vp,
                                              vp, ctypes.POINTER(CTeams), vp, sz, vp]
    L.santapp_build_teams_parents.restype = ctypes.c_int
    L.santapp_build_groups_mean_parents.argtypes = L.santapp_build_teams_parents.argtypes
    L.santapp_build_groups_mean_parents.restype = ctypes.c_int
    L.santapp_decode_workspace_bytes.argtypes = [ctypes.POINTER(CGeom), ctypes.POINTER(CTeams), i32]
    L.santapp_decode_workspace_bytes.restype = sz
    L.santapp_dense_workspace_bytes.argtypes = [ctypes.POINTER(CGeom), ctypes.POINTER(CTeams)]
    L.santapp_dense_workspace_bytes.restype = sz
    L.santapp_decode_attn.argtypes = [ctypes.POINTER(CGeom), ctypes.POINTER(CTeams), vp, vp, vp, vp, i32, i32,
                                      u64, u32, vp, u32, f32, vp, ctypes.POINTER(CDebug), vp, sz, vp]
    L.santapp_set_stage_mask.argtypes = [ctypes.c_int]
    L.santapp_set_stage_mask.restype = None
    L.santapp_decode_attn.restype = ctypes.c_int
    L.santapp_dense_decode_attn.argtypes = [ctypes.POINTER(CGeom), ctypes.POINTER(CTeams), vp, vp, vp, vp, i32,
                                            f32, vp, vp, sz, vp]
    L.santapp_dense_decode_attn.restype = ctypes.c_int
    L.santapp_dense_decode_attn_noalloc.argtypes = [ctypes.POINTER(CGeom), ctypes.POINTER(CTeams), vp, vp, vp, vp,
                                                    i32, f32, vp, vp]
    L.santapp_dense_decode_attn_noalloc.restype = ctypes.c_int
    LG, LT = ctypes.POINTER(CLatentGeom), ctypes.POINTER(CLatentTeams)
    L.santapp_latent_sizes.argtypes = [LG, ctypes.POINTER(i32), ctypes.POINTER(CSizes)]
    L.santapp_latent_sizes.restype = ctypes.c_int
    L.santapp_latent_build_teams.argtypes = [LG, ctypes.POINTER(i32), vp, LT, vp, sz, vp]
    L.santapp_latent_build_teams.restype = ctypes.c_int
    L.santapp_latent_decode_workspace_bytes.argtypes = [LG, LT, i32, i32]
    L.santapp_latent_decode_workspace_bytes.restype = sz
    L.santapp_latent_dense_workspace_bytes.argtypes = [LG, LT]
    L.santapp_latent_dense_workspace_bytes.restype = sz
    L.santapp_latent_decode_attn.argtypes = [LG, LT, vp, vp, vp, i32, i32, u64, u32, vp, u32, f32, vp,
                                             ctypes.POINTER(CDebug), vp, sz, vp]
    L.santapp_latent_decode_attn.restype = ctypes.c_int
    L.santapp_latent_dense_decode_attn.argtypes = [LG, LT, vp, vp, vp, i32, f32, vp, vp, sz, vp]
    L.santapp_latent_dense_decode_attn.restype = ctypes.c_int
    if path is None:
        _lib = L
    return L


def _check(rc):
    if rc != SANTAPP_OK:
        L = load_library()
        detail = L.santapp_strerror(rc).decode()
        if rc in (SANTAPP_ERR_CUDA, SANTAPP_ERR_STATIC_SCRATCH):
            detail += " — " + L.santapp_last_cuda_error().decode()
        raise SantappError(rc, detail)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise SantappError(SANTAPP_ERR_INVALID_ARG, "tensors must be contiguous CUDA tensors")
    return ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


@dataclass
class Geometry:
    n_seqs: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int = 128
    parent_size: int = 512
    reps_per_parent: int = 32
    elem_type: int = 0               # SANTAPP_BF16; 1 = SANTAPP_FP16

    def c(self) -> CGeom:
        return CGeom(self.n_seqs, self.n_q_heads, self.n_kv_heads, self.head_dim, self.parent_size,
                     self.reps_per_parent, self.elem_type)

    @property
    def torch_dtype(self):
        return torch.float16 if self.elem_type == SANTAPP_FP16 else torch.bfloat16


@dataclass
class Sizes:
    rows_total: int
    teams_total: int
    max_teams_per_seq: int
    max_rows_per_seq: int
    team_row_start_elems: int
    build_workspace_bytes: int


class Teams:
    """Team records of one layer: device tensors plus the C struct that points at them."""

    def __init__(self, geom: Geometry, sizes: Sizes, device):
        d = geom.head_dim
        kv = geom.n_kv_heads
        self.geom = geom
        self.sizes = sizes
        self.k_packed = torch.empty((kv, sizes.rows_total, d), dtype=geom.torch_dtype, device=device)
        self.v_packed = torch.empty_like(self.k_packed)
        self.rep_keys = torch.empty((kv, sizes.teams_total, d), dtype=geom.torch_dtype, device=device)
        self.team_row_start = torch.empty((kv, sizes.teams_total + geom.n_seqs), dtype=torch.int32, device=device)
        self.row_token = torch.empty((kv, sizes.rows_total), dtype=torch.int32, device=device)
        self.seq_row_off = torch.empty(geom.n_seqs + 1, dtype=torch.int64, device=device)
        self.seq_team_off = torch.empty(geom.n_seqs + 1, dtype=torch.int64, device=device)
        self.rep_abs_max = torch.empty((kv, geom.n_seqs), dtype=torch.float32, device=device)
        self.team_count = torch.empty((kv, geom.n_seqs), dtype=torch.int32, device=device)
        self.c = CTeams(self.k_packed.data_ptr(), self.v_packed.data_ptr(), self.rep_keys.data_ptr(),
                        self.team_row_start.data_ptr(), self.row_token.data_ptr(),
                        self.seq_row_off.data_ptr(), self.seq_team_off.data_ptr(), self.rep_abs_max.data_ptr(),
                        self.team_count.data_ptr(), sizes.rows_total, sizes.teams_total, sizes.max_teams_per_seq, sizes.max_rows_per_seq)


def santapp_version() -> int:
    return load_library().santapp_version()


def santapp_last_launch_count() -> int:
    return load_library().santapp_last_launch_count()


def santapp_set_stage_mask(mask: int) -> None:
    load_library().santapp_set_stage_mask(mask)


def santapp_build_teams_sizes(geom: Geometry, prompt_len) -> Sizes:
    L = load_library()
    n = len(prompt_len)
    arr = (ctypes.c_int32 * n)(*[int(x) for x in prompt_len])
    out = CSizes()
    g = geom.c()
    _check(L.santapp_build_teams_sizes(ctypes.byref(g), arr, ctypes.byref(out)))
    return Sizes(out.rows_total, out.teams_total, out.max_teams_per_seq, out.max_rows_per_seq,
                 out.team_row_start_elems, out.build_workspace_bytes)


def santapp_build_groups_mean(geom: Geometry, prompt_len, k_prompt: torch.Tensor, v_prompt: torch.Tensor,
                              stream=None) -> Teams:
    """Centroid-guided grouping: one group per contiguous parent, routed by its mean key
    (geom.reps_per_parent must be 1). Arguments as for santapp_build_teams."""
    return santapp_build_teams(geom, prompt_len, k_prompt, v_prompt, stream, _entry="santapp_build_groups_mean")


def santapp_build_teams(geom: Geometry, prompt_len, k_prompt: torch.Tensor, v_prompt: torch.Tensor,
                        stream=None, _entry: str = "santapp_build_teams") -> Teams:
    """k_prompt, v_prompt: bf16 CUDA tensors [n_kv_heads, rows_total, d] in token order."""
    L = load_library()
    sizes = santapp_build_teams_sizes(geom, prompt_len)
    teams = Teams(geom, sizes, k_prompt.device)
    ws = torch.empty(max(sizes.build_workspace_bytes, 256), dtype=torch.uint8, device=k_prompt.device)
    n = len(prompt_len)
    arr = (ctypes.c_int32 * n)(*[int(x) for x in prompt_len])
    g = geom.c()
    _check(getattr(L, _entry)(ctypes.byref(g), arr, _ptr(k_prompt), _ptr(v_prompt), ctypes.byref(teams.c),
                              _ptr(ws), ws.numel(), _stream_ptr(stream)))
    teams._build_ws = ws      # keep alive until the stream has consumed it
    return teams


def _i32_array(values):
    return (ctypes.c_int32 * len(values))(*[int(x) for x in values])


def santapp_kmeans_parent_count(prompt_len: int, parent_size: int) -> int:
    """First line of Algorithm 3: min(N, max(2, N // P)); 0 for N < 2 or P < 1."""
    return int(load_library().santapp_kmeans_parent_count(int(prompt_len), int(parent_size)))


def santapp_kmeans_fit(geom: Geometry, prompt_len, n_centres, k_prompt: torch.Tensor, batch_size: int = 4096,
                       max_iter: int = 100, patience: int = 10, reassignment_ratio: float = 0.01, seed: int = 0,
                       stream_base: int = 0, stream=None, no_host_poll: bool = False):
    """Minibatch k-means fit per (sequence, KV head); the defaults are the paper's settings.
    Returns (centres fp32 [n_kv_heads, sum(n_centres), d], steps int32 [n_kv_heads, n_seqs])."""
    L = load_library()
    g = geom.c()
    o = CKmeansOpts(batch_size, max_iter, patience, 1 if no_host_poll else 0, reassignment_ratio, seed, stream_base, 0)
    n, c = _i32_array(prompt_len), _i32_array(n_centres)
    need = int(L.santapp_kmeans_fit_workspace_bytes(ctypes.byref(g), n, c, ctypes.byref(o)))
    if need == 0:
        raise SantappError(SANTAPP_ERR_INVALID_ARG, "k-means fit arguments")
    dev = k_prompt.device
    ws = torch.empty(need, dtype=torch.uint8, device=dev)
    centres = torch.empty((geom.n_kv_heads, int(sum(n_centres)), geom.head_dim), dtype=torch.float32, device=dev)
    steps = torch.zeros((geom.n_kv_heads, geom.n_seqs), dtype=torch.int32, device=dev)
    _check(L.santapp_kmeans_fit(ctypes.byref(g), n, c, _ptr(k_prompt), ctypes.byref(o), _ptr(centres), _ptr(steps),
                                _ptr(ws), ws.numel(), _stream_ptr(stream)))
    centres._ws = ws
    return centres, steps


def santapp_assign_parents(geom: Geometry, prompt_len, n_centres, k_prompt: torch.Tensor, centres: torch.Tensor,
                           stream=None) -> torch.Tensor:
    """Nearest-centre label of every token. centres: fp32 CUDA tensor [n_kv_heads, sum(n_centres), d].
    Returns int32 [n_kv_heads, rows_total]."""
    L = load_library()
    g = geom.c()
    if centres.dtype != torch.float32:
        raise SantappError(SANTAPP_ERR_INVALID_ARG, "centres must be float32")
    parent_of = torch.empty((geom.n_kv_heads, k_prompt.shape[1]), dtype=torch.int32, device=k_prompt.device)
    ws = torch.empty(max(int(L.santapp_assign_parents_workspace_bytes(ctypes.byref(g))), 256), dtype=torch.uint8,
                     device=k_prompt.device)
    _check(L.santapp_assign_parents(ctypes.byref(g), _i32_array(prompt_len), _i32_array(n_centres), _ptr(k_prompt),
                                    _ptr(centres), _ptr(parent_of), _ptr(ws), ws.numel(), _stream_ptr(stream)))
    parent_of._ws = ws
    return parent_of


def santapp_parent_teams_sizes(geom: Geometry, prompt_len, n_parents) -> Sizes:
    L = load_library()
    out = CSizes()
    g = geom.c()
    _check(L.santapp_parent_teams_sizes(ctypes.byref(g), _i32_array(prompt_len), _i32_array(n_parents),
                                        ctypes.byref(out)))
    return Sizes(out.rows_total, out.teams_total, out.max_teams_per_seq, out.max_rows_per_seq,
                 out.team_row_start_elems, out.build_workspace_bytes)


def santapp_build_groups_mean_parents(geom: Geometry, prompt_len, n_parents, k_prompt: torch.Tensor,
                                      v_prompt: torch.Tensor, parent_of: torch.Tensor, stream=None) -> Teams:
    """Centroid-guided groups on a given partition (geom.reps_per_parent must be 1)."""
    return santapp_build_teams_parents(geom, prompt_len, n_parents, k_prompt, v_prompt, parent_of, stream,
                                       _entry="santapp_build_groups_mean_parents")


def santapp_build_teams_parents(geom: Geometry, prompt_len, n_parents, k_prompt: torch.Tensor,
                                v_prompt: torch.Tensor, parent_of: torch.Tensor, stream=None,
                                _entry: str = "santapp_build_teams_parents") -> Teams:
    """Team records from a parent label per token (int32 CUDA tensor [n_kv_heads, rows_total])."""
    L = load_library()
    sizes = santapp_parent_teams_sizes(geom, prompt_len, n_parents)
    teams = Teams(geom, sizes, k_prompt.device)
    ws = torch.empty(max(sizes.build_workspace_bytes, 256), dtype=torch.uint8, device=k_prompt.device)
    g = geom.c()
    if parent_of.dtype != torch.int32:
        raise SantappError(SANTAPP_ERR_INVALID_ARG, "parent_of must be int32")
    _check(getattr(L, _entry)(ctypes.byref(g), _i32_array(prompt_len), _i32_array(n_parents),
                              _ptr(k_prompt), _ptr(v_prompt), _ptr(parent_of), ctypes.byref(teams.c),
                              _ptr(ws), ws.numel(), _stream_ptr(stream)))
    teams._build_ws = ws      # keep alive until the stream has consumed it
    return teams


def santapp_decode_workspace_bytes(geom: Geometry, teams: Teams, n_sample: int) -> int:
    g = geom.c()
    return int(load_library().santapp_decode_workspace_bytes(ctypes.byref(g), ctypes.byref(teams.c), n_sample))


def santapp_dense_workspace_bytes(geom: Geometry, teams: Teams) -> int:
    g = geom.c()
    return int(load_library().santapp_dense_workspace_bytes(ctypes.byref(g), ctypes.byref(teams.c)))


class DebugBuffers:
    """Optional per-step diagnostics (device tensors)."""

    def __init__(self, geom: Geometry, n_sample: int, device, trace: bool = False):
        B, Hq, Hkv = geom.n_seqs, geom.n_q_heads, geom.n_kv_heads
        self.trace = torch.zeros((5, 256, 16), dtype=torch.int64, device=device) if trace else None
        self.sel_idx = torch.full((B, Hq, n_sample), -1, dtype=torch.int32, device=device)
        self.sel_logc = torch.zeros((B, Hq, n_sample), dtype=torch.float32, device=device)
        self.tau = torch.zeros((B, Hq), dtype=torch.float64, device=device)
        self.union_rows = torch.zeros((B, Hkv), dtype=torch.int32, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.c = CDebug(self.sel_idx.data_ptr(), self.sel_logc.data_ptr(), self.tau.data_ptr(),
                        self.union_rows.data_ptr(), self.status.data_ptr(),
                        self.trace.data_ptr() if trace else None)


def santapp_decode_attn(geom: Geometry, teams: Teams, q: torch.Tensor, k_suffix: Optional[torch.Tensor],
                        v_suffix: Optional[torch.Tensor], suffix_len: Optional[torch.Tensor], n_sample: int,
                        seed: int, step: int, stream_base: int = 0, scale: float = 0.0,
                        out: Optional[torch.Tensor] = None, debug: Optional[DebugBuffers] = None,
                        workspace: Optional[torch.Tensor] = None, stream=None,
                        step_dev: Optional[torch.Tensor] = None) -> torch.Tensor:
    """q bf16 [B, Hq, d]; k_suffix/v_suffix bf16 [B, Hkv, cap, d]; suffix_len int32 [B] (device);
    step_dev optional device int32/uint32 [1] added to `step` on the device."""
    L = load_library()
    if out is None:
        out = torch.empty((geom.n_seqs, geom.n_q_heads, geom.head_dim), dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = torch.empty(santapp_decode_workspace_bytes(geom, teams, n_sample), dtype=torch.uint8,
                                device=q.device)
    cap = 0 if k_suffix is None else int(k_suffix.shape[2])
    g = geom.c()
    _check(L.santapp_decode_attn(ctypes.byref(g), ctypes.byref(teams.c), _ptr(q), _ptr(k_suffix), _ptr(v_suffix),
                                 _ptr(suffix_len), cap, n_sample, ctypes.c_uint64(seed), step, _ptr(step_dev),
                                 stream_base, scale, _ptr(out), ctypes.byref(debug.c) if debug is not None else None,
                                 _ptr(workspace), workspace.numel(), _stream_ptr(stream)))
    return out


def santapp_dense_decode_attn(geom: Geometry, teams: Teams, q: torch.Tensor, k_suffix: Optional[torch.Tensor],
                              v_suffix: Optional[torch.Tensor], suffix_len: Optional[torch.Tensor],
                              scale: float = 0.0, out: Optional[torch.Tensor] = None,
                              workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    L = load_library()
    if out is None:
        out = torch.empty((geom.n_seqs, geom.n_q_heads, geom.head_dim), dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = torch.empty(santapp_dense_workspace_bytes(geom, teams), dtype=torch.uint8, device=q.device)
    cap = 0 if k_suffix is None else int(k_suffix.shape[2])
    g = geom.c()
    _check(L.santapp_dense_decode_attn(ctypes.byref(g), ctypes.byref(teams.c), _ptr(q), _ptr(k_suffix),
                                       _ptr(v_suffix), _ptr(suffix_len), cap, scale, _ptr(out), _ptr(workspace),
                                       workspace.numel(), _stream_ptr(stream)))
    return out


def santapp_dense_decode_attn_noalloc(geom: Geometry, teams: Teams, q: torch.Tensor,
                                      k_suffix: Optional[torch.Tensor], v_suffix: Optional[torch.Tensor],
                                      suffix_len: Optional[torch.Tensor], scale: float = 0.0,
                                      out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Dense decode attention that takes no workspace: for callers that cannot allocate device
    memory around the call, the scratch lives in a fixed array inside the library. Pass `out` to
    keep the call itself free of any allocation; if it is omitted this wrapper (not the library)
    creates the output tensor. Same result as santapp_dense_decode_attn. Calls share the array,
    so do not let two of them overlap on the GPU; the first call on a device should come
    before any stream capture."""
    L = load_library()
    if out is None:
        out = torch.empty((geom.n_seqs, geom.n_q_heads, geom.head_dim), dtype=torch.float32, device=q.device)
    cap = 0 if k_suffix is None else int(k_suffix.shape[2])
    g = geom.c()
    _check(L.santapp_dense_decode_attn_noalloc(ctypes.byref(g), ctypes.byref(teams.c), _ptr(q), _ptr(k_suffix),
                                               _ptr(v_suffix), _ptr(suffix_len), cap, scale, _ptr(out),
                                               _stream_ptr(stream)))
    return out


# ------------------------------------------------------------------------------------------------
# Shared-latent rows (include/santapp_latent.h)
# ------------------------------------------------------------------------------------------------
@dataclass
class LatentGeometry:
    n_seqs: int
    n_heads: int = 16
    parent_size: int = 16
    reps_per_parent: int = 4

    def c(self) -> CLatentGeom:
        return CLatentGeom(self.n_seqs, self.n_heads, self.parent_size, self.reps_per_parent)


class LatentTeams:
    """Team records of shared-latent rows: device tensors plus the C struct that points at them."""

    def __init__(self, geom: LatentGeometry, sizes: Sizes, device):
        self.geom = geom
        self.sizes = sizes
        self.rows_packed = torch.empty((sizes.rows_total, LATENT_ROW), dtype=torch.bfloat16, device=device)
        self.rep_rows = torch.empty((sizes.teams_total, LATENT_ROW), dtype=torch.bfloat16, device=device)
        self.team_row_start = torch.empty(sizes.teams_total + geom.n_seqs, dtype=torch.int32, device=device)
        self.row_token = torch.empty(sizes.rows_total, dtype=torch.int32, device=device)
        self.seq_row_off = torch.empty(geom.n_seqs + 1, dtype=torch.int64, device=device)
        self.seq_team_off = torch.empty(geom.n_seqs + 1, dtype=torch.int64, device=device)
        self.rep_abs_max = torch.empty(geom.n_seqs, dtype=torch.float32, device=device)
        self.c = CLatentTeams(self.rows_packed.data_ptr(), self.rep_rows.data_ptr(), self.team_row_start.data_ptr(),
                              self.row_token.data_ptr(), self.seq_row_off.data_ptr(), self.seq_team_off.data_ptr(),
                              self.rep_abs_max.data_ptr(), sizes.rows_total, sizes.teams_total,
                              sizes.max_teams_per_seq, sizes.max_rows_per_seq)


def santapp_latent_sizes(geom: LatentGeometry, prompt_len) -> Sizes:
    L = load_library()
    out = CSizes()
    g = geom.c()
    _check(L.santapp_latent_sizes(ctypes.byref(g), _i32_array(prompt_len), ctypes.byref(out)))
    return Sizes(out.rows_total, out.teams_total, out.max_teams_per_seq, out.max_rows_per_seq,
                 out.team_row_start_elems, out.build_workspace_bytes)


def santapp_latent_build_teams(geom: LatentGeometry, prompt_len, rows_prompt: torch.Tensor, stream=None) -> LatentTeams:
    """rows_prompt: bf16 CUDA tensor [rows_total, 576] in token order (512 latent values, 64 rotary)."""
    L = load_library()
    sizes = santapp_latent_sizes(geom, prompt_len)
    teams = LatentTeams(geom, sizes, rows_prompt.device)
    ws = torch.empty(max(sizes.build_workspace_bytes, 256), dtype=torch.uint8, device=rows_prompt.device)
    g = geom.c()
    _check(L.santapp_latent_build_teams(ctypes.byref(g), _i32_array(prompt_len), _ptr(rows_prompt), ctypes.byref(teams.c),
                                        _ptr(ws), ws.numel(), _stream_ptr(stream)))
    teams._build_ws = ws
    return teams


def santapp_latent_decode_workspace_bytes(geom: LatentGeometry, teams: LatentTeams, n_sample: int, suffix_cap: int) -> int:
    g = geom.c()
    return int(load_library().santapp_latent_decode_workspace_bytes(ctypes.byref(g), ctypes.byref(teams.c), n_sample,
                                                                    suffix_cap))


def santapp_latent_dense_workspace_bytes(geom: LatentGeometry, teams: LatentTeams) -> int:
    g = geom.c()
    return int(load_library().santapp_latent_dense_workspace_bytes(ctypes.byref(g), ctypes.byref(teams.c)))


class LatentDebugBuffers(DebugBuffers):
    """Diagnostics of a shared-latent step: per (sequence, head) samples, per sequence union rows."""

    def __init__(self, geom: LatentGeometry, n_sample: int, device):
        super().__init__(Geometry(geom.n_seqs, geom.n_heads, 1), n_sample, device)


def santapp_latent_decode_attn(geom: LatentGeometry, teams: LatentTeams, q: torch.Tensor,
                               suffix_rows: Optional[torch.Tensor], suffix_len: Optional[torch.Tensor], n_sample: int,
                               seed: int, step: int, scale: float, stream_base: int = 0,
                               out: Optional[torch.Tensor] = None, debug: Optional[DebugBuffers] = None,
                               workspace: Optional[torch.Tensor] = None, stream=None,
                               step_dev: Optional[torch.Tensor] = None) -> torch.Tensor:
    """q bf16 [B, H, 576]; suffix_rows bf16 [B, cap, 576]; suffix_len int32 [B] (device). Returns fp32 [B, H, 512]."""
    L = load_library()
    cap = 0 if suffix_rows is None else int(suffix_rows.shape[1])
    if out is None:
        out = torch.empty((geom.n_seqs, geom.n_heads, LATENT_DIM), dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = torch.empty(santapp_latent_decode_workspace_bytes(geom, teams, n_sample, cap), dtype=torch.uint8,
                                device=q.device)
    g = geom.c()
    _check(L.santapp_latent_decode_attn(ctypes.byref(g), ctypes.byref(teams.c), _ptr(q), _ptr(suffix_rows),
                                        _ptr(suffix_len), cap, n_sample, ctypes.c_uint64(seed), step, _ptr(step_dev),
                                        stream_base, scale, _ptr(out),
                                        ctypes.byref(debug.c) if debug is not None else None, _ptr(workspace),
                                        workspace.numel(), _stream_ptr(stream)))
    return out


def santapp_latent_dense_decode_attn(geom: LatentGeometry, teams: LatentTeams, q: torch.Tensor,
                                     suffix_rows: Optional[torch.Tensor], suffix_len: Optional[torch.Tensor],
                                     scale: float, out: Optional[torch.Tensor] = None,
                                     workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    L = load_library()
    cap = 0 if suffix_rows is None else int(suffix_rows.shape[1])
    if out is None:
        out = torch.empty((geom.n_seqs, geom.n_heads, LATENT_DIM), dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = torch.empty(santapp_latent_dense_workspace_bytes(geom, teams), dtype=torch.uint8, device=q.device)
    g = geom.c()
    _check(L.santapp_latent_dense_decode_attn(ctypes.byref(g), ctypes.byref(teams.c), _ptr(q), _ptr(suffix_rows),
                                              _ptr(suffix_len), cap, scale, _ptr(out), _ptr(workspace),
                                              workspace.numel(), _stream_ptr(stream)))
    return out


def bf16_bits_to_cuda(bits, device="cuda", dtype=torch.bfloat16):
    """numpy uint16 bit patterns -> CUDA tensor of the 16-bit `dtype` (no value conversion)."""
    import numpy as np
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(dtype)
