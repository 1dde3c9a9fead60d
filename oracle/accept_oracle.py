"""ctypes wrapper of the plain C acceptance oracle (accept_oracle.c).

TEST INFRASTRUCTURE ONLY.  The C file is compiled with gcc on first use (or by
`build_c_oracle()`); nothing here touches CUDA.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "accept_oracle.c")
_LIB = os.path.join(_HERE, "_build", "liboracle_accept.so")
_lib = None


def build_c_oracle(force: bool = False) -> str:
    """Compile accept_oracle.c into a shared library next to it; returns the path."""
    os.makedirs(os.path.dirname(_LIB), exist_ok=True)
    stale = force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if stale:
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build_c_oracle())
        i32p = ctypes.POINTER(ctypes.c_int)
        f32p = ctypes.POINTER(ctypes.c_float)
        f64p = ctypes.POINTER(ctypes.c_double)
        L.radar_oracle_accept_stochastic.restype = ctypes.c_int
        L.radar_oracle_accept_stochastic.argtypes = [
            ctypes.c_int, ctypes.c_int, ctypes.c_int, i32p, i32p, f32p, f32p, i32p, f32p,
            ctypes.c_float, ctypes.c_double, i32p, i32p, i32p, i32p, f64p, f64p]
        L.radar_oracle_accept_length_distribution.restype = ctypes.c_int
        L.radar_oracle_accept_length_distribution.argtypes = [
            ctypes.c_int, ctypes.c_int, ctypes.c_int, i32p, i32p, i32p, f32p, f32p, i32p,
            ctypes.c_double, f64p, f64p]
        _lib = L
    return _lib


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def verify_stochastic(target_logits, draft_logits, tree, u_accept, u_sample, temperature, t_max):
    """Multi-draft recursive rejection sampling over one sequence's tree.

    target_logits [>=n_nodes,V], draft_logits [R,V] float32; tree as returned by
    radar_oracle.rerank_build_tree (uses n_nodes, tok, parent, draft_row);
    u_accept [64] float32, u_sample float.  See accept_oracle.c for the rule.
    """
    n = int(tree["n_nodes"])
    tl = np.ascontiguousarray(target_logits[:n], np.float32)
    dl = np.ascontiguousarray(draft_logits, np.float32)
    V = tl.shape[1]
    tok = np.ascontiguousarray(tree["tok"][:n], np.int32)
    par = np.ascontiguousarray(tree["parent"][:n], np.int32)
    drow = np.ascontiguousarray(tree["draft_row"][:n], np.int32)
    ua = np.ascontiguousarray(u_accept, np.float32)
    path_nodes = np.zeros(t_max + 1, np.int32)
    path_tokens = np.zeros(t_max + 1, np.int32)
    alen = ctypes.c_int()
    nxt = ctypes.c_int()
    am = ctypes.c_double()
    sm = ctypes.c_double()
    rc = lib().radar_oracle_accept_stochastic(
        V, n, t_max, _p(tok, ctypes.c_int), _p(par, ctypes.c_int), _p(tl, ctypes.c_float),
        _p(dl, ctypes.c_float), _p(drow, ctypes.c_int), _p(ua, ctypes.c_float),
        ctypes.c_float(float(u_sample)), float(temperature), ctypes.byref(alen),
        _p(path_nodes, ctypes.c_int), _p(path_tokens, ctypes.c_int), ctypes.byref(nxt),
        ctypes.byref(am), ctypes.byref(sm))
    if rc != 0:
        raise RuntimeError("oracle accept failed")
    path = [int(x) for x in path_nodes if x >= 0]
    best = -1
    for r in range(int(tree["n_leaves"])):
        if all(tree["retrieve"][r, d] == path[d] for d in range(len(path))):
            best = r
            break
    return {
        "accept_len": alen.value, "path_nodes": path_nodes, "path_tokens": path_tokens,
        "next_token": nxt.value, "best_retrieve_row": best,
        "accept_margin": am.value, "sample_margin": sm.value,
    }


def accept_length_distribution(target_logits, draft_logits, tree, temperature, t_max):
    """d = {p_0 .. p_tmax} of Eq. 11-13 for one tree; also P_acc of every node."""
    n = int(tree["n_nodes"])
    tl = np.ascontiguousarray(target_logits[:n], np.float32)
    dl = np.ascontiguousarray(draft_logits, np.float32)
    V = tl.shape[1]
    tok = np.ascontiguousarray(tree["tok"][:n], np.int32)
    par = np.ascontiguousarray(tree["parent"][:n], np.int32)
    dep = np.ascontiguousarray(tree["depth"][:n], np.int32)
    drow = np.ascontiguousarray(tree["draft_row"][:n], np.int32)
    dist = np.zeros(t_max + 1, np.float64)
    pacc = np.zeros(n, np.float64)
    rc = lib().radar_oracle_accept_length_distribution(
        V, n, t_max, _p(tok, ctypes.c_int), _p(par, ctypes.c_int), _p(dep, ctypes.c_int),
        _p(tl, ctypes.c_float), _p(dl, ctypes.c_float), _p(drow, ctypes.c_int), float(temperature),
        _p(dist, ctypes.c_double), _p(pacc, ctypes.c_double))
    if rc != 0:
        raise RuntimeError("oracle distribution failed")
    return dist, pacc
