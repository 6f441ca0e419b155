"""Python access to the CPU oracle (test infrastructure; see iodf_oracle.cpp).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package. It
compiles `iodf_oracle.cpp` with g++ on first use and marshals a model dict (as produced by
`iodf_synth`) into the oracle's own flat descriptor.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "iodf_oracle.cpp")
_LIB = os.path.join(_HERE, "libiodf_oracle.so")
_lib = None


_RANS_SRC = os.path.join(_HERE, "rans_oracle.cpp")
_RANS_LIB = os.path.join(_HERE, "librans_oracle.so")
_rans = None


def _compile(src, lib_path, force):
    if force or not os.path.exists(lib_path) or os.path.getmtime(lib_path) < os.path.getmtime(src):
        tmp = lib_path + ".tmp.%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread", "-o", tmp, src])
        os.replace(tmp, lib_path)
    return lib_path


def build(force=False):
    _compile(_RANS_SRC, _RANS_LIB, force)
    return _compile(_SRC, _LIB, force)


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.orc_rq.restype = ctypes.c_int64
        L.orc_rq.argtypes = [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32]
        _lib = L
    return _lib


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


class Packed:
    """A model dict flattened into the oracle's descriptor, weight and parameter arrays."""

    def __init__(self, model):
        desc, wts, par = [], [], []
        woff = poff = 0

        def layer(ly):
            nonlocal woff, poff
            w = np.ascontiguousarray(ly["w"], dtype=np.int8)
            assert w.shape == (ly["c_out"], ly["k"], ly["k"], ly["c_in"])
            cl = ly["clamp"]
            gate = ly.get("gate")
            desc.extend([ly["k"], ly["c_in"], ly["c_out"], int(ly["relu"]), int(cl is not None),
                         cl[0] if cl else 0, cl[1] if cl else 0, int(gate is not None), woff, poff])
            wts.append(w.reshape(-1))
            woff += w.size
            blk = [ly["bias"], ly["m0"], ly["s"]] + ([gate] if gate is not None else [])
            for a in blk:
                par.append(np.asarray(a, dtype=np.int32).reshape(-1))
                poff += ly["c_out"]

        desc.extend([0x10DF, model["in_c"], model["in_h"], model["in_w"], len(model["levels"])])
        for lv in model["levels"]:
            desc.extend([len(lv["couplings"]), int(lv["split"]), int(lv["prior"] is not None)])
            for cp in lv["couplings"]:
                desc.append(len(cp["perm"]))
                desc.extend(int(v) for v in cp["perm"])
                blocks = cp.get("blocks") or []
                desc.extend([cp["in_m0"], cp["in_s"], len(cp["layers"]), len(blocks)])
                for ly in cp["layers"]:
                    layer(ly)
                for rb in blocks:
                    desc.extend([rb["short_m0"], rb["short_s"], rb["clamp"][0], rb["clamp"][1], len(rb["idx"])])
                    desc.extend(int(v) for v in rb["idx"])
            if lv["prior"] is not None:
                hd = lv["prior"]
                desc.extend([hd["in_m0"], hd["in_s"]])
                layer(hd["layer"])
                desc.extend([hd["ls_lo"], hd["ls_hi"]])
        self.desc = np.array(desc, dtype=np.int32)
        self.wts = np.concatenate(wts) if wts else np.zeros(1, np.int8)
        self.par = np.concatenate(par) if par else np.zeros(1, np.int32)
        self.in_shape = (model["in_c"], model["in_h"], model["in_w"])
        d, df = ctypes.c_long(), ctypes.c_long()
        rc = lib().orc_layout(_p(self.desc), ctypes.c_long(len(self.desc)), _p(self.wts), _p(self.par),
                              ctypes.byref(d), ctypes.byref(df))
        if rc != 0:
            raise ValueError("oracle rejected the model descriptor (rc=%d)" % rc)
        self.d, self.d_fact = d.value, df.value

    def _head(self):
        return (_p(self.desc), ctypes.c_long(len(self.desc)), _p(self.wts), _p(self.par))


def _threads(threads):
    return int(threads or os.cpu_count() or 1)


def forward(pk, x_u8, want_prior=True, threads=None):
    """x_u8 uint8 [B, C, H, W] -> (z int32 [B, d], prior int32 [B, 2, d_fact] | None)."""
    x = np.ascontiguousarray(x_u8, dtype=np.uint8)
    B = x.shape[0]
    assert x.shape[1:] == pk.in_shape
    z = np.empty((B, pk.d), dtype=np.int32)
    prior = np.empty((B, 2, pk.d_fact), dtype=np.int32) if (want_prior and pk.d_fact) else None
    rc = lib().orc_forward(*pk._head(), _p(x), B, _p(z), _p(prior) if prior is not None else None,
                           _threads(threads))
    if rc != 0:
        raise RuntimeError("oracle forward failed (rc=%d)" % rc)
    return z, prior


def inverse(pk, z, want_prior=True, threads=None):
    """z int32 [B, d] -> (x_u8 [B,C,H,W], x_i32 [B,C,H,W], prior | None, out_of_range_count)."""
    z = np.ascontiguousarray(z, dtype=np.int32)
    B = z.shape[0]
    assert z.shape[1] == pk.d
    xu = np.empty((B,) + pk.in_shape, dtype=np.uint8)
    xi = np.empty((B,) + pk.in_shape, dtype=np.int32)
    prior = np.empty((B, 2, pk.d_fact), dtype=np.int32) if (want_prior and pk.d_fact) else None
    oor = ctypes.c_uint32(0)
    rc = lib().orc_inverse(*pk._head(), _p(z), B, _p(xu), _p(xi), _p(prior) if prior is not None else None,
                           ctypes.byref(oor), _threads(threads))
    if rc != 0:
        raise RuntimeError("oracle inverse failed (rc=%d)" % rc)
    return xu, xi, prior, oor.value


def trace(pk, x_u8_one, level, coupling, shape):
    """Flow variable [C, H, W] of one image right after `coupling` of `level`."""
    x = np.ascontiguousarray(x_u8_one, dtype=np.uint8)
    v = np.empty(shape, dtype=np.int32)
    rc = lib().orc_trace(*pk._head(), _p(x), level, coupling, _p(v))
    if rc != 0:
        raise RuntimeError("oracle trace failed (rc=%d)" % rc)
    return v


def rq(a, m0, s):
    return int(lib().orc_rq(int(a), int(m0), int(s)))


def conv_acc(w, bias, x):
    """w int8 [c_out,k,k,c_in], bias int32 [c_out], x int32 [c_in,h,w] -> int64 [c_out,h,w]."""
    w = np.ascontiguousarray(w, dtype=np.int8)
    bias = np.ascontiguousarray(bias, dtype=np.int32)
    x = np.ascontiguousarray(x, dtype=np.int32)
    c_out, k, _, c_in = w.shape
    out = np.empty((c_out,) + x.shape[1:], dtype=np.int64)
    rc = lib().orc_conv_acc(k, c_in, c_out, _p(w), _p(bias), _p(x), x.shape[1], x.shape[2], _p(out))
    if rc != 0:
        raise RuntimeError("accumulator left the int32 range")
    return out


def squeeze(x):
    x = np.ascontiguousarray(x, dtype=np.int32)
    c, h, w = x.shape
    y = np.empty((c * 4, h // 2, w // 2), dtype=np.int32)
    lib().orc_squeeze(_p(x), c, h, w, _p(y))
    return y


def unsqueeze(y):
    y = np.ascontiguousarray(y, dtype=np.int32)
    c4, h2, w2 = y.shape
    x = np.empty((c4 // 4, h2 * 2, w2 * 2), dtype=np.int32)
    lib().orc_unsqueeze(_p(y), c4, h2, w2, _p(x))
    return x


# ---- entropy-coding side (rans_oracle.cpp) ---------------------------------------------------------
def _rans_lib():
    global _rans
    if _rans is None:
        build()
        L = ctypes.CDLL(_RANS_LIB)
        L.orc_rans_cum.restype = ctypes.c_uint32
        L.orc_rans_encode_stream.restype = ctypes.c_long
        _rans = L
    return _rans


def _codec_args(codec):
    G = np.ascontiguousarray(codec["G"], dtype=np.uint16)
    R = np.ascontiguousarray(codec["R"], dtype=np.uint32)
    return G, R, (_p(G), ctypes.c_int(codec["umax"]), _p(R), ctypes.c_int(len(R)))


def rans_cum(codec, ls, k):
    """Cumulative count Cum(k) of scale index ls, k in [0, 4097]."""
    G, R, a = _codec_args(codec)
    return int(_rans_lib().orc_rans_cum(*a, ctypes.c_int(ls), ctypes.c_int(k)))


def rans_encode_stream(codec, z, mu, ls):
    """One stream: per-element int32 arrays in forward order -> uint16 words."""
    G, R, a = _codec_args(codec)
    z, mu, ls = (np.ascontiguousarray(v, dtype=np.int32) for v in (z, mu, ls))
    cap = 3 * len(z) + 2
    words = np.zeros(cap, dtype=np.uint16)
    n = _rans_lib().orc_rans_encode_stream(*a, _p(z), _p(mu), _p(ls), ctypes.c_long(len(z)), _p(words),
                                           ctypes.c_long(cap))
    if n < 0:
        raise RuntimeError("oracle rANS encode failed (rc=%d)" % n)
    return words[:n].copy()


def rans_decode_stream(codec, words, mu, ls):
    G, R, a = _codec_args(codec)
    words = np.ascontiguousarray(words, dtype=np.uint16)
    mu, ls = (np.ascontiguousarray(v, dtype=np.int32) for v in (mu, ls))
    z = np.zeros(len(mu), dtype=np.int32)
    rc = _rans_lib().orc_rans_decode_stream(*a, _p(words), ctypes.c_long(len(words)), _p(mu), _p(ls),
                                            ctypes.c_long(len(mu)), _p(z))
    if rc != 0:
        raise RuntimeError("oracle rANS decode failed (rc=%d)" % rc)
    return z


def rans_blocks(model):
    """[(z offset, elements, prior offset or -1)] per coded block of one image: every factored-out
    block in z order, then the final block."""
    blocks, zo, po = [], 0, 0
    c = model["in_c"]
    for lv in model["levels"]:
        c, px = lv["c"], lv["h"] * lv["w"]
        if lv["split"]:
            n = (c - c // 2) * px
            blocks.append((zo, n, po if lv["prior"] is not None else -1))
            zo += n
            if lv["prior"] is not None:
                po += n
            c = c // 2
    last = model["levels"][-1]
    blocks.append((zo, c * last["h"] * last["w"], -1))
    return blocks


def _rans_batch_args(codec, model):
    blocks = rans_blocks(model)
    E = codec["elems_per_stream"]
    zoff = np.array([b[0] for b in blocks], dtype=np.int64)
    bn = np.array([b[1] for b in blocks], dtype=np.int64)
    poff = np.array([b[2] for b in blocks], dtype=np.int64)
    n_streams = int(sum((n + E - 1) // E for n in bn))
    cap = 3 * E + 2
    return blocks, E, zoff, bn, poff, n_streams, cap


def rans_encode(codec, model, z, prior):
    """z int32 [B,d], prior int32 [B,2,d_fact] (or None) -> (words uint16 [B,S,cap], counts uint32 [B,S])."""
    G, R, a = _codec_args(codec)
    blocks, E, zoff, bn, poff, S, cap = _rans_batch_args(codec, model)
    z = np.ascontiguousarray(z, dtype=np.int32)
    B, d = z.shape
    d_fact = 0 if prior is None else prior.shape[2]
    pr = np.zeros((B, 2, max(d_fact, 1)), np.int32) if prior is None else np.ascontiguousarray(prior, dtype=np.int32)
    words = np.zeros((B, S, cap), dtype=np.uint16)
    counts = np.zeros((B, S), dtype=np.uint32)
    cl = ctypes.c_long
    rc = _rans_lib().orc_rans_encode(*a, ctypes.c_int(codec["final_ls"]), cl(E), _p(z), _p(pr), cl(B), cl(d),
                                     cl(d_fact), ctypes.c_int(len(blocks)), _p(zoff), _p(bn), _p(poff), cl(S),
                                     cl(cap), _p(words), _p(counts))
    if rc != 0:
        raise RuntimeError("oracle rANS encode failed (rc=%d)" % rc)
    return words, counts


def rans_decode_block(codec, model, words, counts, prior, block, z):
    """Decode coded block `block` of every image into z (in place)."""
    G, R, a = _codec_args(codec)
    blocks, E, zoff, bn, poff, S, cap = _rans_batch_args(codec, model)
    B, d = z.shape
    d_fact = 0 if prior is None else prior.shape[2]
    pr = np.zeros((B, 2, max(d_fact, 1)), np.int32) if prior is None else np.ascontiguousarray(prior, dtype=np.int32)
    words = np.ascontiguousarray(words, dtype=np.uint16)
    counts = np.ascontiguousarray(counts, dtype=np.uint32)
    assert z.dtype == np.int32 and z.flags.c_contiguous
    cl = ctypes.c_long
    rc = _rans_lib().orc_rans_decode_block(*a, ctypes.c_int(codec["final_ls"]), cl(E), _p(words), _p(counts), _p(pr),
                                           cl(B), cl(d), cl(d_fact), ctypes.c_int(len(blocks)), _p(zoff), _p(bn),
                                           _p(poff), cl(S), cl(cap), ctypes.c_int(block), _p(z))
    if rc != 0:
        raise RuntimeError("oracle rANS decode failed (rc=%d)" % rc)
    return z
