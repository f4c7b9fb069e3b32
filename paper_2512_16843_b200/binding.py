"""ctypes binding of libllmcache.so: the same entry points as include/llmcache.h.

Only argument marshalling lives here.  Device memory and streams come from
PyTorch; every step of the probe runs in the library's CUDA kernels.  If the
shared library is missing or cannot be loaded the import of this module's
functions fails loudly -- there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# LLMCACHE_LIB selects another build of the same library (the range-checking debug build)
LIB_PATH = os.environ.get("LLMCACHE_LIB") or os.path.join(_HERE, "libllmcache.so")

OK = 0
ERR_ARG, ERR_SHAPE, ERR_NOMEM, ERR_CUDA, ERR_STATE, ERR_TIMEOUT, ERR_UNSUPPORTED, ERR_BOUNDS = -1, -2, -3, -4, -5, -6, -7, -8
F32, BF16 = 0, 1
GT, GE = 0, 1
LRU, LRU_STALENESS = 0, 1
EVICT_STALE, EVICT_IDLE, EVICT_ALL, EVICT_SLOTS = 0, 1, 2, 3
(WHAT_FP, WHAT_RB, WHAT_VALID, WHAT_LAST_USE, WHAT_INSERT_TICK, WHAT_HITS, WHAT_RATE,
 WHAT_RATE_EPOCH, WHAT_ACT, WHAT_TICK) = range(10)

EXPORTS = [
    "llmcache_abi_version", "llmcache_strerror", "llmcache_last_cuda_error", "llmcache_bank_bytes", "llmcache_bank_create",
    "llmcache_bank_destroy", "llmcache_fingerprint", "llmcache_probe", "llmcache_probe_fp",
    "llmcache_commit", "llmcache_evict", "llmcache_bank_export", "llmcache_bank_import",
    "llmcache_bank_stats", "llmcache_bank_status", "llmcache_bank_profile", "llmcache_bank_profile_read",
    "llmcache_fingerprint_static", "llmcache_fingerprint_static_error",
    "llmcache_layer_bytes", "llmcache_layer_create", "llmcache_layer_destroy", "llmcache_layer_forward",
    "llmcache_layer_status", "llmcache_infer", "llmcache_divergence_check", "llmcache_probe_simhash",
    "llmcache_pool", "llmcache_fingerprint_pooled", "llmcache_probe_pooled", "llmcache_bank_pool_out",
    "llmcache_infer_pooled", "llmcache_fingerprint_static_status", "llmcache_bank_debug_knobs",
    "llmcache_layer_debug_knobs", "llmcache_debug_bounds_build", "llmcache_bank_input_stable",
    "llmcache_shard_scan", "llmcache_shard_decide", "llmcache_embed",
]
KNOB_PRODUCER_IDLE = 1
FINGERPRINT_STATIC_MAX_FLOATS = 2 * 1024 * 1024
KERNEL_NAMES = ["pool", "project", "rownorm", "scan", "decide", "touch", "gather", "select", "scatter", "evict",
                "pool_finish"]


class BankDesc(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("device", C.c_int32),
        ("capacity", C.c_uint32), ("seq_len", C.c_uint32), ("d_model", C.c_uint32), ("fp_dim", C.c_uint32),
        ("hidden_dtype", C.c_uint32), ("act_rows", C.c_uint32), ("max_batch", C.c_uint32),
        ("tau", C.c_float), ("cmp", C.c_uint32), ("policy", C.c_uint32),
        ("half_life_ticks", C.c_uint32), ("stale_floor_q8", C.c_uint32),
        ("min_age_ticks", C.c_uint32), ("max_idle_ticks", C.c_uint32), ("store_act", C.c_uint32),
        ("fused_pool", C.c_uint32),
        ("proj", C.c_void_p), ("center", C.c_void_p), ("arena", C.c_void_p), ("arena_bytes", C.c_size_t),
    ]


class ProbeIO(C.Structure):
    _fields_ = [
        ("hit", C.c_void_p), ("slot", C.c_void_p), ("score", C.c_void_p), ("hit_idx", C.c_void_p),
        ("miss_idx", C.c_void_p), ("counts", C.c_void_p), ("counts_host", C.c_void_p),
        ("fp", C.c_void_p), ("rq", C.c_void_p), ("h_miss", C.c_void_p), ("generation", C.c_uint64),
    ]


class LayerDesc(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("device", C.c_int32), ("d_model", C.c_uint32), ("heads", C.c_uint32),
        ("ffn", C.c_uint32), ("seq_len", C.c_uint32), ("max_seqs", C.c_uint32), ("pre_ln", C.c_uint32),
        ("causal", C.c_uint32), ("tanh_gelu", C.c_uint32), ("eps", C.c_float),
        ("w_qkv", C.c_void_p), ("b_qkv", C.c_void_p), ("w_o", C.c_void_p), ("b_o", C.c_void_p),
        ("ln1_g", C.c_void_p), ("ln1_b", C.c_void_p), ("w_1", C.c_void_p), ("b_1", C.c_void_p),
        ("w_2", C.c_void_p), ("b_2", C.c_void_p), ("ln2_g", C.c_void_p), ("ln2_b", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
    ]


WEIGHT_NAMES = ("w_qkv", "b_qkv", "w_o", "b_o", "ln1_g", "ln1_b", "w_1", "b_1", "w_2", "b_2", "ln2_g", "ln2_b")


class Stats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("probes", "sequences", "hits", "misses", "degenerate",
                                          "inserts", "evictions", "dropped", "flushed", "resident",
                                          "kernel_launches")]


class LLMCacheError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = lib().llmcache_last_cuda_error().decode() if status == ERR_CUDA else ""
        super().__init__(f"{where}: {strerror(status)} ({status}) {detail}")


_lib = None


def lib():
    """The loaded shared library (loads it on first use)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2512_16843_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, u32, i32p = C.c_void_p, C.c_uint32, C.c_void_p
        L.llmcache_abi_version.restype = C.c_uint32
        L.llmcache_abi_version.argtypes = []
        L.llmcache_strerror.restype = C.c_char_p
        L.llmcache_strerror.argtypes = [C.c_int]
        L.llmcache_last_cuda_error.restype = C.c_char_p
        L.llmcache_last_cuda_error.argtypes = []
        L.llmcache_embed.argtypes = [vp, C.c_uint64, u32, u32, C.c_int64, vp, vp, C.c_int32, vp, vp, C.c_float, vp, vp, vp]
        L.llmcache_bank_bytes.argtypes = [C.POINTER(BankDesc), C.POINTER(C.c_size_t)]
        L.llmcache_bank_create.argtypes = [C.POINTER(BankDesc), C.POINTER(vp)]
        L.llmcache_bank_destroy.argtypes = [vp]
        L.llmcache_fingerprint.argtypes = [vp, vp, u32, vp, vp, vp]
        L.llmcache_probe.argtypes = [vp, vp, u32, C.c_float, vp, C.POINTER(ProbeIO), vp]
        L.llmcache_probe_fp.argtypes = [vp, vp, u32, C.c_float, vp, C.POINTER(ProbeIO), vp]
        L.llmcache_probe_simhash.argtypes = [vp, vp, u32, C.c_float, vp, C.POINTER(ProbeIO), vp]
        L.llmcache_commit.argtypes = [vp, vp, C.POINTER(ProbeIO), vp, i32p, vp]
        L.llmcache_evict.argtypes = [vp, u32, vp, u32, vp, vp]
        L.llmcache_bank_export.argtypes = [vp, u32, vp, C.c_size_t, vp]
        L.llmcache_bank_import.argtypes = [vp, u32, vp, C.c_size_t, vp]
        L.llmcache_bank_stats.argtypes = [vp, C.POINTER(Stats)]
        L.llmcache_bank_status.argtypes = [vp]
        L.llmcache_bank_profile.argtypes = [vp, C.c_int]
        L.llmcache_bank_profile_read.argtypes = [vp, u32, C.POINTER(C.c_double), C.POINTER(C.c_uint64)]
        L.llmcache_layer_bytes.argtypes = [C.POINTER(LayerDesc), C.POINTER(C.c_size_t)]
        L.llmcache_layer_create.argtypes = [C.POINTER(LayerDesc), C.POINTER(vp)]
        L.llmcache_layer_destroy.argtypes = [vp]
        L.llmcache_layer_forward.argtypes = [vp, vp, u32, vp, vp, vp]
        L.llmcache_layer_status.argtypes = [vp]
        L.llmcache_infer.argtypes = [C.POINTER(vp), C.POINTER(vp), u32, vp, u32, C.c_float, vp, vp, vp, vp,
                                     C.POINTER(ProbeIO), C.POINTER(vp), vp]
        L.llmcache_divergence_check.argtypes = [vp, vp, vp, C.POINTER(ProbeIO), u32, C.c_float, vp, vp, vp, vp, vp]
        L.llmcache_pool.argtypes = [vp, vp, u32, vp, u32, vp]
        L.llmcache_fingerprint_pooled.argtypes = [vp, vp, u32, u32, vp, vp, vp]
        L.llmcache_probe_pooled.argtypes = [vp, vp, u32, vp, u32, C.c_float, vp, C.POINTER(ProbeIO), vp]
        L.llmcache_bank_pool_out.argtypes = [vp, vp, u32]
        L.llmcache_infer_pooled.argtypes = [C.POINTER(vp), C.POINTER(vp), u32, vp, u32, C.c_float, vp, vp, vp, vp,
                                            C.POINTER(ProbeIO), vp, C.POINTER(vp), vp]
        L.llmcache_fingerprint_static.argtypes = [vp, u32, u32, u32, u32, u32, vp, vp, vp, vp, vp]
        L.llmcache_fingerprint_static_error.restype = C.c_char_p
        L.llmcache_fingerprint_static_error.argtypes = []
        L.llmcache_fingerprint_static_status.argtypes = []
        L.llmcache_debug_bounds_build.argtypes = []
        L.llmcache_bank_input_stable.argtypes = [vp, C.c_int]
        L.llmcache_shard_scan.argtypes = [vp, vp, u32, u32, vp, vp]
        L.llmcache_shard_decide.argtypes = [vp, vp, u32, C.c_float, u32, u32, vp, C.POINTER(ProbeIO), vp]
        L.llmcache_bank_debug_knobs.argtypes = [vp, C.c_uint64, u32]
        L.llmcache_layer_debug_knobs.argtypes = [vp, C.c_uint64, u32]
        for name in EXPORTS:
            if name not in ("llmcache_abi_version", "llmcache_strerror", "llmcache_last_cuda_error",
                            "llmcache_fingerprint_static_error"):
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def strerror(status: int) -> str:
    return lib().llmcache_strerror(int(status)).decode()


def _check(rc: int, where: str):
    if rc != OK:
        raise LLMCacheError(rc, where)


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


# ----------------------------------------------------------------------------
# Entry points, named as in llmcache.h
# ----------------------------------------------------------------------------
def llmcache_abi_version() -> int:
    return int(lib().llmcache_abi_version())


def make_desc(*, device=0, capacity, seq_len, d_model, fp_dim, hidden_dtype=BF16, act_rows=0, max_batch,
              tau=0.9, cmp=GT, policy=LRU_STALENESS, half_life_ticks=0, stale_floor_q8=0, min_age_ticks=0,
              max_idle_ticks=0, store_act=1, fused_pool=0, proj=None, center=None, arena=None, arena_bytes=0) -> BankDesc:
    d = BankDesc()
    d.struct_size = C.sizeof(BankDesc)
    d.device, d.capacity, d.seq_len, d.d_model, d.fp_dim = device, capacity, seq_len, d_model, fp_dim
    d.hidden_dtype, d.act_rows, d.max_batch = hidden_dtype, act_rows, max_batch
    d.tau, d.cmp, d.policy = tau, cmp, policy
    d.half_life_ticks, d.stale_floor_q8 = half_life_ticks, stale_floor_q8
    d.min_age_ticks, d.max_idle_ticks, d.store_act = min_age_ticks, max_idle_ticks, store_act
    d.fused_pool = fused_pool
    d.proj, d.center, d.arena, d.arena_bytes = _ptr(proj), _ptr(center), _ptr(arena), arena_bytes
    return d


def llmcache_bank_bytes(desc: BankDesc) -> int:
    out = C.c_size_t(0)
    _check(lib().llmcache_bank_bytes(C.byref(desc), C.byref(out)), "llmcache_bank_bytes")
    return int(out.value)


def llmcache_bank_create(desc: BankDesc) -> int:
    out = C.c_void_p(None)
    _check(lib().llmcache_bank_create(C.byref(desc), C.byref(out)), "llmcache_bank_create")
    return out.value


def llmcache_bank_destroy(bank: int) -> None:
    _check(lib().llmcache_bank_destroy(bank), "llmcache_bank_destroy")


def llmcache_fingerprint(bank, h_in, B, fp, rq, stream=None) -> None:
    _check(lib().llmcache_fingerprint(bank, _ptr(h_in), B, _ptr(fp), _ptr(rq), _stream(stream)),
           "llmcache_fingerprint")


def llmcache_fingerprint_static(h_in, hidden_dtype, B, seq_len, d_model, fp_dim, proj, center, fp, rq,
                                stream=None) -> None:
    """Fingerprint on the current device without a bank and without any allocation by the library
    (for callers whose device memory is all spoken for).  Raises LLMCacheError with the library's
    explanation when the call is refused, e.g. because the batch exceeds the fixed scratch."""
    rc = lib().llmcache_fingerprint_static(_ptr(h_in), hidden_dtype, B, seq_len, d_model, fp_dim, _ptr(proj),
                                           _ptr(center), _ptr(fp), _ptr(rq), _stream(stream))
    if rc != OK:
        err = LLMCacheError(rc, "llmcache_fingerprint_static")
        err.args = (err.args[0] + " " + lib().llmcache_fingerprint_static_error().decode(),)
        raise err


def llmcache_probe(bank, h_in, B, tau, h_out, io: ProbeIO, stream=None) -> None:
    tau = float("nan") if tau is None else tau
    _check(lib().llmcache_probe(bank, _ptr(h_in), B, tau, _ptr(h_out), C.byref(io), _stream(stream)),
           "llmcache_probe")


def llmcache_probe_simhash(bank, h_in, B, tau, h_out, io: ProbeIO, stream=None) -> None:
    tau = float("nan") if tau is None else tau
    _check(lib().llmcache_probe_simhash(bank, _ptr(h_in), B, tau, _ptr(h_out), C.byref(io), _stream(stream)),
           "llmcache_probe_simhash")


def llmcache_probe_fp(bank, h_in, B, tau, h_out, io: ProbeIO, stream=None) -> None:
    tau = float("nan") if tau is None else tau
    _check(lib().llmcache_probe_fp(bank, _ptr(h_in), B, tau, _ptr(h_out), C.byref(io), _stream(stream)),
           "llmcache_probe_fp")


def llmcache_pool(bank, h_in, B, pooled, ld, stream=None) -> None:
    _check(lib().llmcache_pool(bank, _ptr(h_in), B, _ptr(pooled), ld, _stream(stream)), "llmcache_pool")


def llmcache_fingerprint_pooled(bank, pooled, ld, B, fp, rq, stream=None) -> None:
    _check(lib().llmcache_fingerprint_pooled(bank, _ptr(pooled), ld, B, _ptr(fp), _ptr(rq), _stream(stream)),
           "llmcache_fingerprint_pooled")


def llmcache_probe_pooled(bank, pooled, ld, h_in, B, tau, h_out, io: ProbeIO, stream=None) -> None:
    tau = float("nan") if tau is None else tau
    _check(lib().llmcache_probe_pooled(bank, _ptr(pooled), ld, _ptr(h_in), B, tau, _ptr(h_out), C.byref(io),
                                       _stream(stream)), "llmcache_probe_pooled")


def llmcache_bank_pool_out(bank, pooled_out, ld) -> None:
    _check(lib().llmcache_bank_pool_out(bank, _ptr(pooled_out), ld), "llmcache_bank_pool_out")


def llmcache_commit(bank, miss_out, io: ProbeIO, h_out, new_slot, stream=None) -> None:
    _check(lib().llmcache_commit(bank, _ptr(miss_out), C.byref(io), _ptr(h_out), _ptr(new_slot), _stream(stream)),
           "llmcache_commit")


def llmcache_evict(bank, mode, slots=None, n=0, n_evicted_dev=None, stream=None) -> None:
    _check(lib().llmcache_evict(bank, mode, _ptr(slots), n, _ptr(n_evicted_dev), _stream(stream)), "llmcache_evict")


def llmcache_bank_export(bank, what, ptr, nbytes, stream=None) -> None:
    _check(lib().llmcache_bank_export(bank, what, _ptr(ptr), nbytes, _stream(stream)), "llmcache_bank_export")


def llmcache_bank_import(bank, what, ptr, nbytes, stream=None) -> None:
    _check(lib().llmcache_bank_import(bank, what, _ptr(ptr), nbytes, _stream(stream)), "llmcache_bank_import")


def llmcache_bank_stats(bank) -> dict:
    s = Stats()
    _check(lib().llmcache_bank_stats(bank, C.byref(s)), "llmcache_bank_stats")
    return {n: int(getattr(s, n)) for n, _ in Stats._fields_}


def llmcache_bank_status(bank) -> int:
    return int(lib().llmcache_bank_status(bank))


def llmcache_bank_debug_knobs(bank, wait_limit_ns: int, flags: int) -> None:
    _check(lib().llmcache_bank_debug_knobs(bank, wait_limit_ns, flags), "llmcache_bank_debug_knobs")


def llmcache_layer_debug_knobs(layer, wait_limit_ns: int, flags: int) -> None:
    _check(lib().llmcache_layer_debug_knobs(layer, wait_limit_ns, flags), "llmcache_layer_debug_knobs")


def llmcache_debug_bounds_build() -> bool:
    return bool(lib().llmcache_debug_bounds_build())


def llmcache_fingerprint_static_status() -> int:
    return int(lib().llmcache_fingerprint_static_status())


def llmcache_shard_scan(bank, fp, B, slot_base, words, stream=None) -> None:
    _check(lib().llmcache_shard_scan(bank, _ptr(fp), B, slot_base, _ptr(words), _stream(stream)), "llmcache_shard_scan")


def llmcache_shard_decide(bank, words, B, tau, slot_base, n_total, h_out, io: ProbeIO, stream=None) -> None:
    tau = float("nan") if tau is None else tau
    _check(lib().llmcache_shard_decide(bank, _ptr(words), B, tau, slot_base, n_total, _ptr(h_out), C.byref(io),
                                       _stream(stream)), "llmcache_shard_decide")


def llmcache_bank_profile(bank, enable: bool) -> None:
    _check(lib().llmcache_bank_profile(bank, 1 if enable else 0), "llmcache_bank_profile")


def llmcache_bank_profile_read(bank, kernel_id: int):
    ms, n = C.c_double(0.0), C.c_uint64(0)
    _check(lib().llmcache_bank_profile_read(bank, kernel_id, C.byref(ms), C.byref(n)), "llmcache_bank_profile_read")
    return float(ms.value), int(n.value)


# ----------------------------------------------------------------------------
# Buffer holders (allocation and marshalling only)
# ----------------------------------------------------------------------------
class ProbeBuffers:
    """Device buffers for one probe of up to B sequences, plus the C struct that points at them."""

    def __init__(self, B: int, fp_dim: int, device="cuda", pinned_counts: bool = True,
                 h_miss: Optional[torch.Tensor] = None):
        dev = torch.device(device)
        Bm = max(B, 1)
        self.B = B
        self.hit = torch.zeros(Bm, dtype=torch.uint8, device=dev)
        self.slot = torch.full((Bm,), -1, dtype=torch.int32, device=dev)
        self.score = torch.zeros(Bm, dtype=torch.float32, device=dev)
        self.hit_idx = torch.zeros(Bm, dtype=torch.int32, device=dev)
        self.miss_idx = torch.zeros(Bm, dtype=torch.int32, device=dev)
        self.counts = torch.zeros(2, dtype=torch.int32, device=dev)
        self.counts_host = torch.zeros(2, dtype=torch.int32).pin_memory() if pinned_counts else None
        self.fp = torch.zeros((Bm, fp_dim), dtype=torch.bfloat16, device=dev)
        self.rq = torch.zeros(Bm, dtype=torch.float32, device=dev)
        self.new_slot = torch.full((Bm,), -1, dtype=torch.int32, device=dev)
        self.h_miss = h_miss
        self.io = ProbeIO()
        self.io.hit, self.io.slot, self.io.score = self.hit.data_ptr(), self.slot.data_ptr(), self.score.data_ptr()
        self.io.hit_idx, self.io.miss_idx = self.hit_idx.data_ptr(), self.miss_idx.data_ptr()
        self.io.counts = self.counts.data_ptr()
        self.io.counts_host = self.counts_host.data_ptr() if pinned_counts else None
        self.io.fp, self.io.rq = self.fp.data_ptr(), self.rq.data_ptr()
        self.io.h_miss = h_miss.data_ptr() if h_miss is not None else None
        self.io.generation = 0


_WHAT_DTYPE = {
    WHAT_FP: torch.bfloat16, WHAT_RB: torch.float32, WHAT_VALID: torch.uint8, WHAT_LAST_USE: torch.int32,
    WHAT_INSERT_TICK: torch.int32, WHAT_HITS: torch.int32, WHAT_RATE: torch.int32, WHAT_RATE_EPOCH: torch.int32,
    WHAT_ACT: torch.bfloat16,
}


class Bank:
    """Owner of one llmcache_bank_t handle (one transformer layer's cache)."""

    def __init__(self, **kw):
        self._proj = kw.get("proj")
        self._center = kw.get("center")
        self.desc = make_desc(**kw)
        self.handle = llmcache_bank_create(self.desc)
        self.N, self.n, self.d, self.k = self.desc.capacity, self.desc.seq_len, self.desc.d_model, self.desc.fp_dim
        self.act_rows = self.desc.act_rows or self.desc.capacity
        self.device = torch.device("cuda", self.desc.device)

    def close(self):
        if getattr(self, "handle", None):
            llmcache_bank_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _shape(self, what):
        if what == WHAT_FP:
            return (self.N, self.k)
        if what == WHAT_ACT:
            return (self.act_rows, self.n * self.d)
        return (self.N,)

    def export(self, what) -> torch.Tensor:
        """Copy of one bank array as a host tensor (synchronises)."""
        if what == WHAT_TICK:
            t = torch.zeros(1, dtype=torch.int64)
            llmcache_bank_export(self.handle, what, t.data_ptr(), 8)
            return t
        dev = torch.empty(self._shape(what), dtype=_WHAT_DTYPE[what], device=self.device)
        llmcache_bank_export(self.handle, what, dev.data_ptr(), dev.numel() * dev.element_size())
        torch.cuda.synchronize(self.device)
        return dev.cpu()

    def import_(self, what, t: torch.Tensor):
        if what == WHAT_TICK:
            t = t.to(torch.int64).contiguous()
            llmcache_bank_import(self.handle, what, t.data_ptr(), 8)
            return
        t = t.to(device=self.device).contiguous()
        llmcache_bank_import(self.handle, what, t.data_ptr(), t.numel() * t.element_size())
        torch.cuda.synchronize(self.device)

    def probe(self, h_in, bufs: ProbeBuffers, h_out=None, tau=None, B=None, stream=None):
        B = h_in.shape[0] if B is None else B
        llmcache_probe(self.handle, h_in, B, tau, h_out, bufs.io, stream)

    def probe_pooled(self, pooled, bufs: ProbeBuffers, B, h_out=None, tau=None, h_in=None, stream=None):
        llmcache_probe_pooled(self.handle, pooled, pooled.stride(0), h_in, B, tau, h_out, bufs.io, stream)

    def pool_out(self, pooled_out):
        """Position means of the rows written by the next probes + commits go to pooled_out [B, >=d] f32
        (None switches it off)."""
        llmcache_bank_pool_out(self.handle, pooled_out, 0 if pooled_out is None else pooled_out.stride(0))
        self._pool_out = pooled_out

    def pool(self, h_in, pooled, B=None, stream=None):
        llmcache_pool(self.handle, h_in, h_in.shape[0] if B is None else B, pooled, pooled.stride(0), stream)

    def fingerprint_pooled(self, pooled, fp, rq, B=None, stream=None):
        llmcache_fingerprint_pooled(self.handle, pooled, pooled.stride(0), pooled.shape[0] if B is None else B,
                                    fp, rq, stream)

    def probe_fp(self, bufs: ProbeBuffers, B, h_out=None, tau=None, h_in=None, stream=None):
        llmcache_probe_fp(self.handle, h_in, B, tau, h_out, bufs.io, stream)

    def commit(self, miss_out, bufs: ProbeBuffers, h_out=None, stream=None):
        llmcache_commit(self.handle, miss_out, bufs.io, h_out, bufs.new_slot, stream)

    def evict(self, mode, slots: Optional[torch.Tensor] = None, count: Optional[torch.Tensor] = None, stream=None):
        n = 0 if slots is None else slots.numel()
        llmcache_evict(self.handle, mode, slots, n, count, stream)

    def stats(self) -> dict:
        return llmcache_bank_stats(self.handle)

    def status(self) -> int:
        return llmcache_bank_status(self.handle)

    def debug_knobs(self, wait_limit_ns: int = 0, flags: int = 0):
        llmcache_bank_debug_knobs(self.handle, wait_limit_ns, flags)

    def input_stable(self, stable: bool = True):
        """Promise that probe inputs are never written by the kernel preceding the probe in its stream."""
        _check(lib().llmcache_bank_input_stable(self.handle, 1 if stable else 0), "llmcache_bank_input_stable")

    def profile(self, enable: bool):
        llmcache_bank_profile(self.handle, enable)

    def profile_read(self) -> dict:
        """{kernel name: (total ms, launches)} since the last read."""
        return {name: llmcache_bank_profile_read(self.handle, i) for i, name in enumerate(KERNEL_NAMES)}


# ----------------------------------------------------------------------------
# Miss-path transformer layer and the layer-wise caching loop
# ----------------------------------------------------------------------------
def llmcache_layer_bytes(desc: LayerDesc) -> int:
    out = C.c_size_t(0)
    _check(lib().llmcache_layer_bytes(C.byref(desc), C.byref(out)), "llmcache_layer_bytes")
    return int(out.value)


def llmcache_layer_create(desc: LayerDesc) -> int:
    out = C.c_void_p(None)
    _check(lib().llmcache_layer_create(C.byref(desc), C.byref(out)), "llmcache_layer_create")
    return out.value


def llmcache_layer_destroy(layer: int) -> None:
    _check(lib().llmcache_layer_destroy(layer), "llmcache_layer_destroy")


def llmcache_layer_forward(layer, x, n_seqs, n_seqs_dev, out, stream=None) -> None:
    _check(lib().llmcache_layer_forward(layer, _ptr(x), n_seqs, _ptr(n_seqs_dev), _ptr(out), _stream(stream)),
           "llmcache_layer_forward")


def llmcache_layer_status(layer) -> int:
    return int(lib().llmcache_layer_status(layer))


def llmcache_embed(tokens, tok_emb, pos_emb, h0, *, layer_norm=True, ln_gain=None, ln_bias=None, eps=1e-5,
                   bad_ids=None, stream=None) -> None:
    """h0 = E(X) of Algorithm 1: token + position embeddings, optionally layer-normed.  tokens: int64 [S, n] on the
    device; tok_emb bf16 [vocab, d]; pos_emb bf16 [n, d] or None; h0 bf16 [S, n, d]."""
    S, n = tokens.shape
    vocab, d = tok_emb.shape
    _check(lib().llmcache_embed(_ptr(tokens), S, n, d, vocab, _ptr(tok_emb), _ptr(pos_emb), int(layer_norm),
                                _ptr(ln_gain), _ptr(ln_bias), eps, _ptr(h0), _ptr(bad_ids), _stream(stream)),
           "llmcache_embed")


def llmcache_infer(banks, layers, h0, B, tau, buf_a, buf_b, h_miss, miss_out, io, stream=None) -> int:
    """Algorithm 1 over all layers; returns the device address (buf_a or buf_b) that will hold h_L."""
    n = len(layers)
    larr = (C.c_void_p * n)(*layers)
    barr = (C.c_void_p * n)(*banks) if banks is not None else None
    final = C.c_void_p(None)
    tau = float("nan") if tau is None else tau
    _check(lib().llmcache_infer(barr, larr, n, _ptr(h0), B, tau, _ptr(buf_a), _ptr(buf_b), _ptr(h_miss),
                                _ptr(miss_out), C.byref(io) if io is not None else None, C.byref(final),
                                _stream(stream)), "llmcache_infer")
    return final.value


def llmcache_infer_pooled(banks, layers, h0, B, tau, buf_a, buf_b, h_miss, miss_out, io, pooled, stream=None) -> int:
    """Algorithm 1 with fingerprint-on-write; returns the device address that will hold h_L."""
    n = len(layers)
    larr = (C.c_void_p * n)(*layers)
    barr = (C.c_void_p * n)(*banks)
    final = C.c_void_p(None)
    tau = float("nan") if tau is None else tau
    _check(lib().llmcache_infer_pooled(barr, larr, n, _ptr(h0), B, tau, _ptr(buf_a), _ptr(buf_b), _ptr(h_miss),
                                       _ptr(miss_out), C.byref(io), _ptr(pooled), C.byref(final), _stream(stream)),
           "llmcache_infer_pooled")
    return final.value


def llmcache_divergence_check(bank, layer, h_in, io, stride, bound, h_sample, out_sample, rel_out, counters_dev,
                              stream=None) -> None:
    _check(lib().llmcache_divergence_check(bank, layer, _ptr(h_in), C.byref(io), stride, bound, _ptr(h_sample),
                                           _ptr(out_sample), _ptr(rel_out), _ptr(counters_dev), _stream(stream)),
           "llmcache_divergence_check")


class Layer:
    """Owner of one llmcache_layer_t handle; keeps the weight tensors alive (the library borrows them)."""

    def __init__(self, weights: dict, *, device=0, heads, seq_len, max_seqs, pre_ln=False, causal=False,
                 tanh_gelu=False, eps=1e-5, workspace: Optional[torch.Tensor] = None):
        self.weights = {k: weights[k].contiguous() for k in WEIGHT_NAMES}
        d = LayerDesc()
        d.struct_size = C.sizeof(LayerDesc)
        d.device = device
        d.d_model = self.weights["w_o"].shape[0]
        d.heads, d.ffn, d.seq_len, d.max_seqs = heads, self.weights["w_1"].shape[0], seq_len, max_seqs
        d.pre_ln, d.causal, d.tanh_gelu, d.eps = int(pre_ln), int(causal), int(tanh_gelu), eps
        for k in WEIGHT_NAMES:
            setattr(d, k, self.weights[k].data_ptr())
        self.workspace = workspace
        if workspace is not None:
            d.workspace, d.workspace_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
        self.desc = d
        self.handle = llmcache_layer_create(d)

    def forward(self, x, out, n_seqs=None, n_seqs_dev=None, stream=None):
        llmcache_layer_forward(self.handle, x, x.shape[0] if n_seqs is None else n_seqs, n_seqs_dev, out, stream)

    def status(self) -> int:
        return llmcache_layer_status(self.handle)

    def debug_knobs(self, wait_limit_ns: int = 0, flags: int = 0):
        llmcache_layer_debug_knobs(self.handle, wait_limit_ns, flags)

    def close(self):
        if getattr(self, "handle", None):
            llmcache_layer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
