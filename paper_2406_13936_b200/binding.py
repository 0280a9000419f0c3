"""Thin ctypes binding of the C ABI in include/abs.h.

Argument marshalling only: every function takes torch tensors (device memory) or
plain numbers, passes raw pointers and sizes to the library and raises AbsError on a
non-zero return code.  Nothing is computed here, and there is no fallback: if the
shared library is missing or cannot be loaded the import of a function fails loudly.
"""
import ctypes
import os

import torch

from . import build as _build

ABS_F32, ABS_BF16 = 0, 1
ABS_TEST_NORM, ABS_TEST_AUG_INNER_PRODUCT, ABS_TEST_NORM_WORKERS = 0, 1, 2
STATUS_NONFINITE, STATUS_ZERO_MEAN, STATUS_TIMEOUT, STATUS_NORM_ONLY = 1, 2, 4, 8
STATS_RECORD_BYTES = 56


class AbsError(RuntimeError):
    pass


class TestCfg(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int), ("reserved", ctypes.c_int), ("eta", ctypes.c_double),
                ("theta", ctypes.c_double), ("nu", ctypes.c_double), ("b_max", ctypes.c_longlong),
                ("row_weight", ctypes.c_double), ("divisor", ctypes.c_double)]


class AdamWCfg(ctypes.Structure):
    _fields_ = [("lr", ctypes.c_float), ("beta1", ctypes.c_float), ("beta2", ctypes.c_float),
                ("eps", ctypes.c_float), ("weight_decay", ctypes.c_float), ("reserved", ctypes.c_int),
                ("step", ctypes.c_longlong)]


class Stats(ctypes.Structure):
    _fields_ = [("gbar_sq", ctypes.c_double), ("var_norm", ctypes.c_double), ("var_ip", ctypes.c_double),
                ("var_orth", ctypes.c_double), ("sum_sq", ctypes.c_double), ("rows", ctypes.c_longlong),
                ("status", ctypes.c_uint), ("recomputed", ctypes.c_uint)]


class RoundCtl(ctypes.Structure):
    _fields_ = [("samples", ctypes.c_longlong), ("rounds", ctypes.c_longlong), ("n_stop", ctypes.c_longlong),
                ("reserved", ctypes.c_longlong)]


class RoundOpts(ctypes.Structure):
    _fields_ = [("test_every_step", ctypes.c_int), ("per_worker", ctypes.c_int), ("eta_m", ctypes.c_void_p),
                ("ctl", ctypes.c_void_p)]


class StatsPlan(ctypes.Structure):
    _fields_ = [(name, ctypes.c_int) for name in
                ("route", "lanes_per_row", "warps_per_box", "boxes_per_stage", "stages", "box_rows", "row_boxes",
                 "rows_per_thread", "keep_in_registers", "full", "cluster_size", "rows_per_cta")] + \
               [("stage_bytes", ctypes.c_uint), ("reserved", ctypes.c_uint), ("smem_bytes", ctypes.c_size_t)]


EXPORTS = {
    "abs_plan_stats": [ctypes.c_int, ctypes.c_longlong, ctypes.c_int, ctypes.c_int, ctypes.c_size_t,
                       ctypes.POINTER(StatsPlan)],
    "abs_create": [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int, ctypes.c_size_t],
    "abs_destroy": [ctypes.c_void_p],
    "abs_set_tuning": [ctypes.c_void_p, ctypes.c_char_p, ctypes.c_longlong],
    "abs_test_stats": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_longlong,
                       ctypes.c_longlong, ctypes.c_longlong, ctypes.c_longlong, ctypes.c_void_p,
                       ctypes.c_void_p, ctypes.c_void_p],
    "abs_test_stats_host": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_longlong,
                            ctypes.c_longlong, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                            ctypes.c_void_p],
    "abs_test_stats_noalloc": [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_longlong, ctypes.c_longlong,
                               ctypes.c_longlong, ctypes.c_longlong, ctypes.c_void_p, ctypes.c_void_p,
                               ctypes.c_void_p],
    "abs_next_batch": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(TestCfg),
                       ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p],
    "abs_logreg_grads": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_longlong, ctypes.c_longlong,
                         ctypes.c_void_p, ctypes.c_longlong, ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong,
                         ctypes.c_void_p, ctypes.c_void_p],
    "abs_logreg_round": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_longlong, ctypes.c_longlong,
                         ctypes.c_void_p, ctypes.c_longlong, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                         ctypes.c_longlong, ctypes.c_float, ctypes.POINTER(TestCfg), ctypes.c_void_p, ctypes.c_void_p,
                         ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p],
    "abs_logreg_rounds_fused": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_longlong,
                                ctypes.c_longlong, ctypes.c_void_p, ctypes.c_longlong, ctypes.c_int, ctypes.c_void_p,
                                ctypes.c_int, ctypes.c_int, ctypes.c_float, ctypes.POINTER(TestCfg), ctypes.c_void_p,
                                ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p],
    "abs_logreg_rounds_fused_opts": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_longlong,
                                     ctypes.c_longlong, ctypes.c_void_p, ctypes.c_longlong, ctypes.c_int,
                                     ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_float,
                                     ctypes.POINTER(TestCfg), ctypes.POINTER(RoundOpts), ctypes.c_void_p,
                                     ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p],
    "abs_logreg_round_per_step": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_longlong,
                                  ctypes.c_longlong, ctypes.c_void_p, ctypes.c_longlong, ctypes.c_void_p, ctypes.c_int,
                                  ctypes.c_int, ctypes.POINTER(ctypes.c_longlong), ctypes.c_float,
                                  ctypes.POINTER(TestCfg), ctypes.POINTER(RoundOpts), ctypes.c_void_p, ctypes.c_void_p,
                                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p],
    "abs_mlp_round_per_step": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_longlong,
                               ctypes.POINTER(ctypes.c_int), ctypes.c_void_p, ctypes.c_longlong, ctypes.c_void_p,
                               ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_longlong), ctypes.c_float,
                               ctypes.POINTER(TestCfg), ctypes.POINTER(RoundOpts), ctypes.c_void_p, ctypes.c_size_t,
                               ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p],
    "abs_round_count": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong,
                        ctypes.c_longlong, ctypes.c_void_p],
    "abs_mlp_param_count": [ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_longlong)],
    "abs_mlp_scratch_bytes": [ctypes.c_int, ctypes.c_longlong, ctypes.POINTER(ctypes.c_int),
                              ctypes.POINTER(ctypes.c_size_t)],
    "abs_mlp_grads": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_longlong,
                      ctypes.POINTER(ctypes.c_int), ctypes.c_void_p, ctypes.c_longlong, ctypes.c_void_p, ctypes.c_int,
                      ctypes.c_longlong, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p],
    "abs_mlp_per_sample": [ctypes.c_void_p, ctypes.POINTER(ctypes.c_int), ctypes.c_longlong, ctypes.c_int,
                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_longlong, ctypes.c_void_p],
    "abs_mlp_fused_stats": [ctypes.c_void_p, ctypes.POINTER(ctypes.c_int), ctypes.c_longlong, ctypes.c_int,
                            ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p],
    "abs_mlp_round": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_longlong,
                      ctypes.POINTER(ctypes.c_int), ctypes.c_void_p, ctypes.c_longlong, ctypes.c_void_p, ctypes.c_int,
                      ctypes.c_int, ctypes.c_longlong, ctypes.c_float, ctypes.POINTER(TestCfg), ctypes.c_void_p,
                      ctypes.c_size_t, ctypes.c_void_p, ctypes.c_longlong, ctypes.c_void_p, ctypes.c_void_p,
                      ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p],
    "abs_next_batch_local": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(TestCfg), ctypes.c_void_p,
                             ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p],
    "abs_stats_merge": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong,
                        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p],
    "local_sgd_step": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong,
                       ctypes.c_longlong, ctypes.c_float, ctypes.c_int, ctypes.c_void_p],
    "local_adamw_step": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                         ctypes.c_int, ctypes.c_longlong, ctypes.c_longlong, ctypes.POINTER(AdamWCfg),
                         ctypes.c_int, ctypes.c_void_p],
    "local_shb_step": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                       ctypes.c_longlong, ctypes.c_longlong, ctypes.c_float, ctypes.c_float, ctypes.c_float,
                       ctypes.c_int, ctypes.c_void_p],
    "replica_average": [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong, ctypes.c_longlong,
                        ctypes.c_void_p],
}

_lib = None


def library_path():
    return _build.LIB_PATH


def load_library():
    """dlopen the CUDA library; raises AbsError if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise AbsError("CUDA library %s is missing: run paper_2406_13936_b200.build.build() "
                       "(there is no CPU fallback)" % path)
    lib = ctypes.CDLL(path)
    for name, argtypes in EXPORTS.items():
        fn = getattr(lib, name)
        fn.argtypes = argtypes
        fn.restype = ctypes.c_int
    lib.abs_last_error.argtypes = [ctypes.c_void_p]
    lib.abs_last_error.restype = ctypes.c_char_p
    lib.abs_noalloc_last_error.argtypes = []
    lib.abs_noalloc_last_error.restype = ctypes.c_char_p
    _lib = lib
    return lib


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else ctypes.c_void_p(0)


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _dtype_code(t):
    if t.dtype == torch.float32:
        return ABS_F32
    if t.dtype == torch.bfloat16:
        return ABS_BF16
    raise AbsError("G must be float32 or bfloat16, got %s" % t.dtype)


class Context:
    """Owns an abs_ctx.  One context per device; calls are issued in stream order."""

    def __init__(self, device=0, workspace_bytes=0):
        self._lib = load_library()
        handle = ctypes.c_void_p()
        rc = self._lib.abs_create(ctypes.byref(handle), int(device), int(workspace_bytes))
        if rc != 0:
            raise AbsError("abs_create failed (%d): %s" % (rc, self._lib.abs_last_error(None).decode()))
        self._h = handle
        self.device = int(device)

    def close(self):
        if getattr(self, "_h", None):
            self._lib.abs_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc, what):
        if rc != 0:
            raise AbsError("%s failed (%d): %s" % (what, rc, self._lib.abs_last_error(self._h).decode()))

    def set_tuning(self, key, value):
        self._check(self._lib.abs_set_tuning(self._h, key.encode(), int(value)), "abs_set_tuning")

    # ---- statistics --------------------------------------------------------------------
    def new_stats(self, M):
        """Device buffer for M abs_stats records (M x 7 float64 words)."""
        return torch.zeros((M, 7), dtype=torch.float64, device="cuda:%d" % self.device)

    def abs_test_stats(self, G, stats_out, gbar_out=None, stream=None):
        """G: [M, b, d] or [b, d] device tensor (last dim contiguous); stats_out from new_stats."""
        if G.dim() == 2:
            G = G.unsqueeze(0)
        if G.stride(2) != 1:
            raise AbsError("the last dimension of G must be contiguous")
        M, b, d = G.shape
        rc = self._lib.abs_test_stats(self._h, _ptr(G), _dtype_code(G), M, b, d, G.stride(1), G.stride(0),
                                      _ptr(gbar_out), _ptr(stats_out), _stream(stream))
        self._check(rc, "abs_test_stats")
        return stats_out

    def abs_test_stats_host(self, G_host, want_gbar=False, gbar_dev=None, stats_dev=None, stream=None):
        """G_host: contiguous CPU tensor [M, b, d]; returns (list of stats dicts, gbar or None).
        gbar_dev / stats_dev: optional device tensors that also receive the results."""
        if G_host.dim() == 2:
            G_host = G_host.unsqueeze(0)
        G_host = G_host.contiguous()
        M, b, d = G_host.shape
        recs = (Stats * M)()
        gbar = torch.empty((M, d), dtype=torch.float32) if want_gbar else None
        rc = self._lib.abs_test_stats_host(self._h, _ptr(G_host), _dtype_code(G_host), M, b, d, _ptr(gbar),
                                           ctypes.cast(recs, ctypes.c_void_p), _ptr(gbar_dev), _ptr(stats_dev),
                                           _stream(stream))
        self._check(rc, "abs_test_stats_host")
        return [_record_to_dict(r) for r in recs], gbar

    def abs_next_batch(self, stats, cfg, b_cur, b_next, T_out=None, stream=None):
        """stats: device records; cfg: TestCfg; b_cur / b_next: int64 device tensors of one element."""
        M = stats.shape[0]
        rc = self._lib.abs_next_batch(self._h, _ptr(stats), M, ctypes.byref(cfg), _ptr(b_cur), _ptr(T_out),
                                      _ptr(b_next), _stream(stream))
        self._check(rc, "abs_next_batch")
        return b_next

    def abs_next_batch_local(self, stats, cfg, b_cur, b_next, eta_m=None, T_out=None, stream=None):
        """Per-worker sizes: b_cur / b_next int64 device tensors [M]; eta_m float64 device tensor [M] or None."""
        M = stats.shape[0]
        self._check(self._lib.abs_next_batch_local(self._h, _ptr(stats), M, ctypes.byref(cfg), _ptr(eta_m),
                                                   _ptr(b_cur), _ptr(T_out), _ptr(b_next), _stream(stream)),
                    "abs_next_batch_local")
        return b_next

    def abs_stats_merge(self, mean_a, mean_b, rec_a, rec_b, stream=None):
        """Folds sub-batch (mean_b, rec_b) into the running (mean_a, rec_a); mean tensors [M, d] fp32."""
        M, d = mean_a.shape
        self._check(self._lib.abs_stats_merge(self._h, _ptr(mean_a), _ptr(mean_b), M, d, _ptr(rec_a), _ptr(rec_b),
                                              _stream(stream)), "abs_stats_merge")

    # ---- local updates -------------------------------------------------------------------
    @staticmethod
    def _replicas(X):
        if X.dim() == 1:
            X = X.unsqueeze(0)
        if X.stride(1) != 1:
            raise AbsError("replica tensors must be contiguous in the last dimension")
        return X, X.shape[0], X.shape[1], X.stride(0)

    def local_sgd_step(self, X, Gb, lr, average_after=False, stream=None):
        X2, M, d, stride = self._replicas(X)
        Gb2, _, _, gstride = self._replicas(Gb)
        if gstride != stride and M > 1:
            raise AbsError("X and Gb must share the replica stride")
        self._check(self._lib.local_sgd_step(self._h, _ptr(X2), _ptr(Gb2), M, d, stride, float(lr),
                                             int(bool(average_after)), _stream(stream)), "local_sgd_step")

    def local_adamw_step(self, X, Mom1, Mom2, Gb, cfg, average_after=False, stream=None):
        X2, M, d, stride = self._replicas(X)
        for t in (Mom1, Mom2, Gb):
            if self._replicas(t)[3] != stride and M > 1:
                raise AbsError("all replica tensors must share the replica stride")
        self._check(self._lib.local_adamw_step(self._h, _ptr(X2), _ptr(Mom1), _ptr(Mom2), _ptr(Gb), M, d, stride,
                                               ctypes.byref(cfg), int(bool(average_after)), _stream(stream)),
                    "local_adamw_step")

    def local_shb_step(self, X, Buf, Gb, lr, momentum, weight_decay, average_after=False, stream=None):
        X2, M, d, stride = self._replicas(X)
        for t in (Buf, Gb):
            if self._replicas(t)[3] != stride and M > 1:
                raise AbsError("all replica tensors must share the replica stride")
        self._check(self._lib.local_shb_step(self._h, _ptr(X2), _ptr(Buf), _ptr(Gb), M, d, stride, float(lr),
                                             float(momentum), float(weight_decay), int(bool(average_after)),
                                             _stream(stream)), "local_shb_step")

    # ---- producers and rounds ----------------------------------------------------------------
    def abs_logreg_grads(self, A, y, idx, X, b, G, stream=None):
        """A [n, d], y [n], idx [M, >=b] int32, X [M, d] -> G [M, b, d] (all device tensors)."""
        n, d = A.shape
        M = X.shape[0]
        self._check(self._lib.abs_logreg_grads(self._h, _ptr(A), _ptr(y), n, d, _ptr(idx), idx.stride(0), _ptr(X), M,
                                               int(b), _ptr(G), _stream(stream)), "abs_logreg_grads")

    def abs_logreg_round(self, A, y, idx, X, H, b, lr, cfg, G_scratch, Gb_scratch, stats, b_dev, T_out=None,
                         ctl=None, stream=None):
        """idx [H, M, >=b] int32 (contiguous in H and M); b_dev int64 device tensor holding b; ctl: the
        device counter block from new_round_ctl, or None."""
        n, d = A.shape
        M = X.shape[0]
        self._check(self._lib.abs_logreg_round(self._h, _ptr(A), _ptr(y), n, d, _ptr(idx), idx.stride(1), _ptr(X), M,
                                               int(H), int(b), float(lr), ctypes.byref(cfg), _ptr(G_scratch),
                                               _ptr(Gb_scratch), _ptr(stats), _ptr(T_out), _ptr(b_dev), _ptr(ctl),
                                               _stream(stream)), "abs_logreg_round")

    def new_round_ctl(self, n_stop=0, samples=0, rounds=0):
        """Device counter block (abs_round_ctl) as an int64 tensor [samples, rounds, n_stop, 0]."""
        return torch.tensor([int(samples), int(rounds), int(n_stop), 0], dtype=torch.int64,
                            device="cuda:%d" % self.device)

    def abs_round_count(self, ctl, sizes, times, add_rounds=0, stream=None):
        self._check(self._lib.abs_round_count(self._h, _ptr(ctl), _ptr(sizes), sizes.numel(), int(times),
                                              int(add_rounds), _stream(stream)), "abs_round_count")

    def abs_logreg_round_per_step(self, A, y, idx, X, H, b_sizes, lr, cfg, opts, G_scratch, Gb_scratch, stats,
                                  b_dev, T_out=None, stream=None):
        """The round with the test after every local step.  b_sizes: list of M current sizes; returns the
        list of sizes after the round.  idx [H, M, >= cfg.b_max]; stats from new_stats(H * M);
        T_out [H, M] or None; b_dev int64 device tensor [M]; opts from make_round_opts or None."""
        n, d = A.shape
        M = X.shape[0]
        sizes = (ctypes.c_longlong * M)(*[int(v) for v in b_sizes])
        self._check(self._lib.abs_logreg_round_per_step(
            self._h, _ptr(A), _ptr(y), n, d, _ptr(idx), idx.stride(1), _ptr(X), M, int(H), sizes, float(lr),
            ctypes.byref(cfg), ctypes.byref(opts) if opts is not None else None, _ptr(G_scratch), _ptr(Gb_scratch),
            _ptr(stats), _ptr(T_out), _ptr(b_dev), _stream(stream)), "abs_logreg_round_per_step")
        return list(sizes)

    def abs_mlp_round_per_step(self, inputs_, labels, dims, idx, X, H, b_sizes, lr, cfg, opts, scratch, Gb_scratch,
                               stats, b_dev, T_out=None, stream=None):
        """As abs_logreg_round_per_step for the MLP problem (statistics from activations and deltas)."""
        n = inputs_.shape[0]
        M = X.shape[0]
        sizes = (ctypes.c_longlong * M)(*[int(v) for v in b_sizes])
        self._check(self._lib.abs_mlp_round_per_step(
            self._h, _ptr(inputs_), _ptr(labels), n, (ctypes.c_int * 4)(*dims), _ptr(idx), idx.stride(1), _ptr(X), M,
            int(H), sizes, float(lr), ctypes.byref(cfg), ctypes.byref(opts) if opts is not None else None,
            _ptr(scratch), scratch.numel(), _ptr(Gb_scratch), _ptr(stats), _ptr(T_out), _ptr(b_dev),
            _stream(stream)), "abs_mlp_round_per_step")
        return list(sizes)

    def abs_logreg_rounds_fused(self, A, y, idx, X, H, lr, cfg, stats, b_dev, T_out=None, b_hist=None, stream=None):
        """idx [rounds, H, M, >= cfg.b_max] int32 (contiguous but for the last stride); stats [rounds*M, 7] from
        new_stats(rounds * M); T_out [rounds, M] and b_hist [rounds + 1] int64 or None; b_dev int64 device tensor."""
        n, d = A.shape
        M = X.shape[0]
        rounds = idx.shape[0]
        if idx.dim() != 4 or idx.shape[1] != H or idx.shape[2] != M or idx.stride(3) != 1 or \
                idx.stride(1) != M * idx.stride(2) or idx.stride(0) != H * idx.stride(1):
            raise ValueError("idx must be [rounds, H, M, stride] with the first three dimensions packed")
        if stats.shape[0] < rounds * M:
            raise ValueError("stats needs rounds * M records")
        if not (A.is_contiguous() and X.is_contiguous()):
            raise ValueError("A and X must be contiguous")
        self._check(self._lib.abs_logreg_rounds_fused(self._h, _ptr(A), _ptr(y), n, d, _ptr(idx), idx.stride(2),
                                                      int(rounds), _ptr(X), M, int(H), float(lr), ctypes.byref(cfg),
                                                      _ptr(stats), _ptr(T_out), _ptr(b_hist), _ptr(b_dev),
                                                      _stream(stream)), "abs_logreg_rounds_fused")

    def abs_logreg_rounds_fused_opts(self, A, y, idx, X, H, lr, cfg, opts, stats, b_dev, T_out=None, b_hist=None,
                                     stream=None):
        """The fused rounds with the cadence / size ownership / counters of `opts` (make_round_opts).
        b_dev int64 [M]; with opts.test_every_step: stats from new_stats(rounds * H * M), T_out and b_hist
        [rounds, H, M]; else stats new_stats(rounds * M), T_out and b_hist [rounds, M]."""
        n, d = A.shape
        M = X.shape[0]
        rounds = idx.shape[0]
        if idx.dim() != 4 or idx.shape[1] != H or idx.shape[2] != M or idx.stride(3) != 1 or \
                idx.stride(1) != M * idx.stride(2) or idx.stride(0) != H * idx.stride(1):
            raise ValueError("idx must be [rounds, H, M, stride] with the first three dimensions packed")
        per = H if opts.test_every_step else 1
        if stats.shape[0] < rounds * per * M or b_dev.numel() < M:
            raise ValueError("stats needs rounds * %d * M records and b_dev M entries" % per)
        if not (A.is_contiguous() and X.is_contiguous()):
            raise ValueError("A and X must be contiguous")
        self._check(self._lib.abs_logreg_rounds_fused_opts(
            self._h, _ptr(A), _ptr(y), n, d, _ptr(idx), idx.stride(2), int(rounds), _ptr(X), M, int(H), float(lr),
            ctypes.byref(cfg), ctypes.byref(opts), _ptr(stats), _ptr(T_out), _ptr(b_hist), _ptr(b_dev),
            _stream(stream)), "abs_logreg_rounds_fused_opts")

    def mlp_param_count(self, dims):
        out = ctypes.c_longlong()
        self._check(self._lib.abs_mlp_param_count((ctypes.c_int * 4)(*dims), ctypes.byref(out)), "abs_mlp_param_count")
        return out.value

    def mlp_scratch(self, M, b, dims):
        """Device scratch tensor (uint8) large enough for abs_mlp_grads with M workers and batch size b."""
        out = ctypes.c_size_t()
        self._check(self._lib.abs_mlp_scratch_bytes(int(M), int(b), (ctypes.c_int * 4)(*dims), ctypes.byref(out)),
                    "abs_mlp_scratch_bytes")
        return torch.empty(out.value, dtype=torch.uint8, device="cuda:%d" % self.device)

    def abs_mlp_grads(self, inputs_, labels, dims, idx, X, b, Gb, scratch, stream=None):
        n = inputs_.shape[0]
        M = X.shape[0]
        self._check(self._lib.abs_mlp_grads(self._h, _ptr(inputs_), _ptr(labels), n, (ctypes.c_int * 4)(*dims),
                                            _ptr(idx), idx.stride(0), _ptr(X), M, int(b), _ptr(Gb), _ptr(scratch),
                                            scratch.numel(), _stream(stream)), "abs_mlp_grads")

    def abs_mlp_per_sample(self, dims, b, worker, scratch, G, stream=None):
        """G: [b, row_stride] device tensor view with stride(0) >= d."""
        self._check(self._lib.abs_mlp_per_sample(self._h, (ctypes.c_int * 4)(*dims), int(b), int(worker),
                                                 _ptr(scratch), _ptr(G), G.stride(0), _stream(stream)),
                    "abs_mlp_per_sample")

    def abs_mlp_fused_stats(self, dims, b, scratch, Gb, stats, stream=None):
        """Statistics of all workers from the scratch and the batch gradients of abs_mlp_grads."""
        M = Gb.shape[0]
        self._check(self._lib.abs_mlp_fused_stats(self._h, (ctypes.c_int * 4)(*dims), int(b), M, _ptr(scratch),
                                                  scratch.numel(), _ptr(Gb), _ptr(stats), _stream(stream)),
                    "abs_mlp_fused_stats")

    def abs_mlp_round(self, inputs_, labels, dims, idx, X, H, b, lr, cfg, scratch, G_scratch, g_row_stride,
                      Gb_scratch, stats, b_dev, T_out=None, ctl=None, stream=None):
        n = inputs_.shape[0]
        M = X.shape[0]
        self._check(self._lib.abs_mlp_round(self._h, _ptr(inputs_), _ptr(labels), n, (ctypes.c_int * 4)(*dims),
                                            _ptr(idx), idx.stride(1), _ptr(X), M, int(H), int(b), float(lr),
                                            ctypes.byref(cfg), _ptr(scratch), scratch.numel(), _ptr(G_scratch),
                                            int(g_row_stride), _ptr(Gb_scratch), _ptr(stats), _ptr(T_out),
                                            _ptr(b_dev), _ptr(ctl), _stream(stream)), "abs_mlp_round")

    def replica_average(self, X, stream=None):
        X2, M, d, stride = self._replicas(X)
        self._check(self._lib.replica_average(self._h, _ptr(X2), M, d, stride, _stream(stream)), "replica_average")


def abs_test_stats_noalloc(G, stats_out, gbar_out=None, stream=None):
    """Context-free statistics that allocate nothing (scratch is a fixed array inside the library).

    For callers that may not call cudaMalloc: same arguments and results as
    Context.abs_test_stats, limited to b <= 2048 rows and M <= 64 workers, on the current
    CUDA device.  Calls that may overlap on the GPU must be ordered by the caller.
    """
    lib = load_library()
    if G.dim() == 2:
        G = G.unsqueeze(0)
    if G.stride(2) != 1:
        raise AbsError("the last dimension of G must be contiguous")
    M, b, d = G.shape
    rc = lib.abs_test_stats_noalloc(_ptr(G), _dtype_code(G), M, b, d, G.stride(1), G.stride(0), _ptr(gbar_out),
                                    _ptr(stats_out), _stream(stream))
    if rc != 0:
        raise AbsError("abs_test_stats_noalloc failed (%d): %s" % (rc, lib.abs_noalloc_last_error().decode()))
    return stats_out


def plan_stats(dtype, b, aligned=True, sm_count=148, smem_optin=232448):
    """The kernel and tile shape abs_test_stats would use for b rows of `dtype` ("f32" / "bf16"); needs no GPU."""
    lib = load_library()
    plan = StatsPlan()
    rc = lib.abs_plan_stats({"f32": ABS_F32, "bf16": ABS_BF16}[dtype], int(b), int(bool(aligned)), int(sm_count),
                            int(smem_optin), ctypes.byref(plan))
    if rc != 0:
        raise AbsError("abs_plan_stats failed (%d)" % rc)
    return {name: getattr(plan, name) for name, _ in StatsPlan._fields_ if name != "reserved"}


def _record_to_dict(r):
    return dict(gbar_sq=r.gbar_sq, var_norm=r.var_norm, var_ip=r.var_ip, var_orth=r.var_orth, sum_sq=r.sum_sq,
                rows=r.rows, status=r.status, recomputed=r.recomputed)


def stats_to_dicts(stats):
    """Copy device abs_stats records (tensor from Context.new_stats) to a list of dicts."""
    host = stats.detach().cpu().contiguous()
    raw = host.numpy().tobytes()
    out = []
    for m in range(host.shape[0]):
        out.append(_record_to_dict(Stats.from_buffer_copy(raw[m * STATS_RECORD_BYTES:(m + 1) * STATS_RECORD_BYTES])))
    return out


def make_test_cfg(kind, b_max, eta=0.0, theta=0.0, nu=0.0, row_weight=1.0, divisor=1.0):
    code = {"norm": ABS_TEST_NORM, "aug_ip": ABS_TEST_AUG_INNER_PRODUCT, "norm_workers": ABS_TEST_NORM_WORKERS}[kind]
    return TestCfg(code, 0, float(eta), float(theta), float(nu), int(b_max), float(row_weight), float(divisor))


def make_round_opts(test_every_step=False, per_worker=False, eta_m=None, ctl=None):
    """abs_round_opts; eta_m: float64 device tensor [M] or None; ctl: tensor from Context.new_round_ctl or None.
    The tensors must stay alive while the options are in use."""
    return RoundOpts(int(bool(test_every_step)), int(bool(per_worker)), _ptr(eta_m), _ptr(ctl))


def make_adamw_cfg(lr, beta1, beta2, eps, weight_decay, step):
    return AdamWCfg(float(lr), float(beta1), float(beta2), float(eps), float(weight_decay), 0, int(step))
