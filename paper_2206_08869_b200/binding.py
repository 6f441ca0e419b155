"""ctypes binding of include/iodf.h. Argument marshalling only: model dicts (numpy arrays) become
the C descriptor structs, torch tensors become device pointers, the current torch stream becomes
the cudaStream_t. The function names are those of the C ABI."""
import ctypes as C
import os

import numpy as np

from . import build as _build

IODF_ABI_VERSION = 3
IODF_PLAN_LATENCY, IODF_PLAN_THROUGHPUT = 0, 1
IODF_MAX_LEVELS = 8

DECLARED_SYMBOLS = ["iodf_create", "iodf_destroy", "iodf_get_layout", "iodf_forward", "iodf_inverse",
                    "iodf_inverse_level", "iodf_forward_patches", "iodf_inverse_patches",
                    "iodf_codec_create", "iodf_codec_destroy", "iodf_codec_get_layout", "iodf_rans_encode",
                    "iodf_rans_decode_block", "iodf_codec_check", "iodf_rans_packed_capacity", "iodf_rans_pack",
                    "iodf_rans_unpack", "iodf_compress_host", "iodf_decompress_host",
                    "iodf_forward_host", "iodf_inverse_host", "iodf_forward_timed", "iodf_inverse_timed", "iodf_forward_static",
                    "iodf_static_scratch_bytes_per_image", "iodf_check", "iodf_launches_per_call",
                    "iodf_selftest_timeout", "iodf_int8_mma_peak", "iodf_level_kernel_name",
                    "iodf_level_images_per_cta",
                    "iodf_strerror", "iodf_last_cuda_error"]


class LayerDesc(C.Structure):
    _fields_ = [("k", C.c_uint32), ("c_in", C.c_uint32), ("c_out", C.c_uint32), ("relu", C.c_uint32),
                ("has_clamp", C.c_uint32), ("clamp_lo", C.c_int32), ("clamp_hi", C.c_int32),
                ("weight_off", C.c_uint64), ("requant_off", C.c_uint64)]


class ResBlockDesc(C.Structure):
    _fields_ = [("short_m0", C.c_int32), ("short_s", C.c_int32), ("clamp_lo", C.c_int32), ("clamp_hi", C.c_int32),
                ("n_idx", C.c_uint32), ("idx", C.POINTER(C.c_int32))]


class CouplingDesc(C.Structure):
    _fields_ = [("perm", C.POINTER(C.c_int32)), ("in_m0", C.c_int32), ("in_s", C.c_int32),
                ("n_layers", C.c_uint32), ("layers", C.POINTER(LayerDesc)),
                ("n_blocks", C.c_uint32), ("blocks", C.POINTER(ResBlockDesc))]


class LevelDesc(C.Structure):
    _fields_ = [("n_couplings", C.c_uint32), ("couplings", C.POINTER(CouplingDesc)), ("split", C.c_uint32),
                ("has_prior", C.c_uint32), ("prior_in_m0", C.c_int32), ("prior_in_s", C.c_int32),
                ("prior_layer", LayerDesc), ("ls_lo", C.c_int32), ("ls_hi", C.c_int32)]


class ModelDesc(C.Structure):
    _fields_ = [("abi_version", C.c_uint32), ("in_c", C.c_uint32), ("in_h", C.c_uint32), ("in_w", C.c_uint32),
                ("n_levels", C.c_uint32), ("max_batch", C.c_uint32), ("levels", C.POINTER(LevelDesc)),
                ("plan", C.c_uint32)]


class Layout(C.Structure):
    _fields_ = [("d", C.c_uint64), ("d_fact", C.c_uint64), ("n_levels", C.c_uint32),
                ("level_c", C.c_uint32 * IODF_MAX_LEVELS), ("level_h", C.c_uint32 * IODF_MAX_LEVELS),
                ("level_w", C.c_uint32 * IODF_MAX_LEVELS), ("z_off", C.c_uint64 * IODF_MAX_LEVELS),
                ("prior_off", C.c_uint64 * IODF_MAX_LEVELS), ("z_final_off", C.c_uint64),
                ("macs_per_image", C.c_uint64)]


class CodecDesc(C.Structure):
    _fields_ = [("abi_version", C.c_uint32), ("sigmoid_table", C.c_void_p), ("umax", C.c_uint32),
                ("inv_scale", C.c_void_p), ("n_scales", C.c_uint32), ("final_ls", C.c_int32),
                ("elems_per_stream", C.c_uint32)]


class CodecLayout(C.Structure):
    _fields_ = [("n_blocks", C.c_uint32), ("n_streams", C.c_uint32), ("words_per_stream", C.c_uint32),
                ("block_level", C.c_int32 * (IODF_MAX_LEVELS + 1)), ("block_z_off", C.c_uint64 * (IODF_MAX_LEVELS + 1)),
                ("block_elems", C.c_uint64 * (IODF_MAX_LEVELS + 1)),
                ("block_first_stream", C.c_uint32 * (IODF_MAX_LEVELS + 1)),
                ("block_streams", C.c_uint32 * (IODF_MAX_LEVELS + 1))]


class IodfError(RuntimeError):
    def __init__(self, status, what):
        super().__init__("%s failed: %s (status %d)" % (what, iodf_strerror(status), status))
        self.status = status


_lib = None


def load_library(path=None):
    """Load libiodf_b200.so (building it with nvcc if it is missing or stale). Raises if that is
    impossible: there is no fallback implementation."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    lib_path = path or _build.build()
    if not os.path.exists(lib_path):
        raise RuntimeError("libiodf_b200.so is missing: run paper_2206_08869_b200.build.build()")
    L = C.CDLL(lib_path)
    vp = C.c_void_p
    L.iodf_create.restype = C.c_int
    L.iodf_create.argtypes = [C.POINTER(ModelDesc), vp, C.c_size_t, vp, C.c_size_t, C.c_int, C.POINTER(vp)]
    L.iodf_destroy.restype = None
    L.iodf_destroy.argtypes = [vp]
    L.iodf_get_layout.restype = C.c_int
    L.iodf_get_layout.argtypes = [vp, C.POINTER(Layout)]
    L.iodf_forward.restype = C.c_int
    L.iodf_forward.argtypes = [vp, vp, C.c_int, vp, vp, vp]
    L.iodf_inverse.restype = C.c_int
    L.iodf_inverse.argtypes = [vp, vp, C.c_int, vp, vp, vp, vp]
    L.iodf_inverse_level.restype = C.c_int
    L.iodf_inverse_level.argtypes = [vp, C.c_int, C.c_int, vp, C.c_int, vp, vp, vp, vp]
    L.iodf_forward_patches.restype = C.c_int
    L.iodf_forward_patches.argtypes = [vp, vp, C.c_int, C.c_int, vp, vp, vp]
    L.iodf_inverse_patches.restype = C.c_int
    L.iodf_inverse_patches.argtypes = [vp, vp, C.c_int, C.c_int, vp, vp, vp, vp]
    L.iodf_codec_create.restype = C.c_int
    L.iodf_codec_create.argtypes = [vp, C.POINTER(CodecDesc), C.POINTER(vp)]
    L.iodf_codec_destroy.restype = None
    L.iodf_codec_destroy.argtypes = [vp]
    L.iodf_codec_get_layout.restype = C.c_int
    L.iodf_codec_get_layout.argtypes = [vp, C.POINTER(CodecLayout)]
    L.iodf_rans_encode.restype = C.c_int
    L.iodf_rans_encode.argtypes = [vp, vp, vp, C.c_int, vp, vp, vp]
    L.iodf_rans_decode_block.restype = C.c_int
    L.iodf_rans_decode_block.argtypes = [vp, C.c_int, vp, vp, vp, C.c_int, vp, vp]
    L.iodf_codec_check.restype = C.c_int
    L.iodf_codec_check.argtypes = [vp, vp, C.POINTER(C.c_uint32)]
    L.iodf_rans_packed_capacity.restype = C.c_size_t
    L.iodf_rans_packed_capacity.argtypes = [vp, C.c_int]
    L.iodf_rans_pack.restype = C.c_int
    L.iodf_rans_pack.argtypes = [vp, vp, vp, C.c_int, vp, vp]
    L.iodf_rans_unpack.restype = C.c_int
    L.iodf_rans_unpack.argtypes = [vp, vp, C.c_size_t, C.c_int, vp, vp, vp]
    L.iodf_compress_host.restype = C.c_int
    L.iodf_compress_host.argtypes = [vp, vp, vp, C.c_int, vp, C.c_size_t, C.POINTER(C.c_size_t), vp]
    L.iodf_decompress_host.restype = C.c_int
    L.iodf_decompress_host.argtypes = [vp, vp, vp, C.c_size_t, C.c_int, vp, vp]
    L.iodf_forward_host.restype = C.c_int
    L.iodf_forward_host.argtypes = [vp, vp, C.c_int, vp, vp, vp]
    L.iodf_inverse_host.restype = C.c_int
    L.iodf_inverse_host.argtypes = [vp, vp, C.c_int, vp, vp]
    L.iodf_forward_timed.restype = C.c_int
    L.iodf_forward_timed.argtypes = [vp, vp, C.c_int, vp, vp, vp, C.POINTER(C.c_float)]
    L.iodf_inverse_timed.restype = C.c_int
    L.iodf_inverse_timed.argtypes = [vp, vp, C.c_int, vp, vp, vp, vp, C.POINTER(C.c_float)]
    L.iodf_forward_static.restype = C.c_int
    L.iodf_forward_static.argtypes = [vp, vp, C.c_int, vp, vp, vp]
    L.iodf_static_scratch_bytes_per_image.restype = C.c_size_t
    L.iodf_static_scratch_bytes_per_image.argtypes = [vp]
    L.iodf_check.restype = C.c_int
    L.iodf_check.argtypes = [vp, vp]
    L.iodf_selftest_timeout.restype = C.c_int
    L.iodf_selftest_timeout.argtypes = [vp, C.c_uint32, vp]
    L.iodf_int8_mma_peak.restype = C.c_int
    L.iodf_int8_mma_peak.argtypes = [vp, C.c_uint32, vp, C.POINTER(C.c_ulonglong)]
    L.iodf_level_kernel_name.restype = C.c_char_p
    L.iodf_level_kernel_name.argtypes = [vp, C.c_int]
    L.iodf_level_images_per_cta.restype = C.c_int
    L.iodf_level_images_per_cta.argtypes = [vp, C.c_int]
    L.iodf_launches_per_call.restype = C.c_int
    L.iodf_launches_per_call.argtypes = [vp, C.c_int]
    L.iodf_strerror.restype = C.c_char_p
    L.iodf_strerror.argtypes = [C.c_int]
    L.iodf_last_cuda_error.restype = C.c_int
    L.iodf_last_cuda_error.argtypes = [vp]
    if path is None:
        _lib = L
    return L


def iodf_strerror(status):
    return load_library().iodf_strerror(int(status)).decode()


class _Marshalled:
    """C descriptor structs for a model dict, with every referenced array kept alive."""

    def __init__(self, model, max_batch, plan=0):
        self.keep = []
        wts, par = [], []
        self.woff = self.poff = 0

        def layer(ly):
            w = np.ascontiguousarray(ly["w"], dtype=np.int8)
            cl = ly["clamp"]
            if ly.get("gate") is not None:
                raise ValueError("gated (masked-dense) layers must be compacted before deployment")
            d = LayerDesc(ly["k"], ly["c_in"], ly["c_out"], int(ly["relu"]), int(cl is not None),
                          cl[0] if cl else 0, cl[1] if cl else 0, self.woff, self.poff)
            wts.append(w.reshape(-1))
            self.woff += w.size
            for a in (ly["bias"], ly["m0"], ly["s"]):
                par.append(np.asarray(a, dtype=np.int32).reshape(-1))
                self.poff += ly["c_out"]
            return d

        levels = (LevelDesc * len(model["levels"]))()
        for li, lv in enumerate(model["levels"]):
            cps = (CouplingDesc * max(1, len(lv["couplings"])))()
            for ki, cp in enumerate(lv["couplings"]):
                perm = np.ascontiguousarray(cp["perm"], dtype=np.int32)
                lays = (LayerDesc * len(cp["layers"]))(*[layer(ly) for ly in cp["layers"]])
                self.keep += [perm, lays]
                rblocks = cp.get("blocks") or []
                rbs = (ResBlockDesc * max(1, len(rblocks)))()
                for bi, rb in enumerate(rblocks):
                    idx = np.ascontiguousarray(rb["idx"], dtype=np.int32)
                    self.keep.append(idx)
                    rbs[bi] = ResBlockDesc(rb["short_m0"], rb["short_s"], rb["clamp"][0], rb["clamp"][1], len(idx),
                                           idx.ctypes.data_as(C.POINTER(C.c_int32)))
                self.keep.append(rbs)
                cps[ki] = CouplingDesc(perm.ctypes.data_as(C.POINTER(C.c_int32)), cp["in_m0"], cp["in_s"],
                                       len(cp["layers"]), lays, len(rblocks), rbs)
            self.keep.append(cps)
            levels[li].n_couplings = len(lv["couplings"])
            levels[li].couplings = cps
            levels[li].split = int(lv["split"])
            levels[li].has_prior = int(lv["prior"] is not None)
            if lv["prior"] is not None:
                hd = lv["prior"]
                levels[li].prior_in_m0, levels[li].prior_in_s = hd["in_m0"], hd["in_s"]
                levels[li].prior_layer = layer(hd["layer"])
                levels[li].ls_lo, levels[li].ls_hi = hd["ls_lo"], hd["ls_hi"]
        self.levels = levels
        self.desc = ModelDesc(IODF_ABI_VERSION, model["in_c"], model["in_h"], model["in_w"], len(model["levels"]),
                              int(max_batch), levels, int(plan))
        self.wts = np.concatenate(wts) if wts else np.zeros(1, np.int8)
        self.par = np.concatenate(par) if par else np.zeros(1, np.int32)


class Model:
    """Handle of an iodf_model; destroyed when garbage collected."""

    def __init__(self, handle, layout, in_shape, max_batch):
        self.handle, self.layout, self.in_shape, self.max_batch = handle, layout, in_shape, max_batch
        self.d, self.d_fact = int(layout.d), int(layout.d_fact)

    def __del__(self):
        h, self.handle = getattr(self, "handle", None), None
        if h and _lib is not None:
            _lib.iodf_destroy(h)


def iodf_create(model, max_batch, device=0, marshalled=None, plan=IODF_PLAN_LATENCY):
    """plan: IODF_PLAN_LATENCY (the shortest step) or IODF_PLAN_THROUGHPUT (fewer CTAs per launch, for
    several batches in flight on streams and handles of their own); see include/iodf.h."""
    L = load_library()
    m = marshalled or _Marshalled(model, max_batch, plan)
    out = C.c_void_p()
    rc = L.iodf_create(C.byref(m.desc), m.wts.ctypes.data, m.wts.size, m.par.ctypes.data, m.par.size, int(device),
                       C.byref(out))
    if rc != 0:
        raise IodfError(rc, "iodf_create")
    lay = Layout()
    L.iodf_get_layout(out, C.byref(lay))
    return Model(out, lay, (model["in_c"], model["in_h"], model["in_w"]), int(max_batch))


def iodf_destroy(model):
    h, model.handle = model.handle, None
    if h:
        load_library().iodf_destroy(h)


def iodf_get_layout(model):
    return model.layout


def _stream(stream):
    if stream is None:
        import torch
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)
    return C.c_void_p(int(getattr(stream, "cuda_stream", stream)))    # a torch stream or a raw handle


def _ptr(t):
    return C.c_void_p(0 if t is None else t.data_ptr())


def iodf_forward(model, x_u8, z=None, prior=None, stream=None, want_prior=True):
    """x_u8: cuda uint8 [B,C,H,W]. Returns (z int32 [B,d], prior int32 [B,2,d_fact] | None)."""
    import torch
    B = x_u8.shape[0]
    assert x_u8.is_cuda and x_u8.dtype == torch.uint8 and x_u8.is_contiguous()
    if z is None:
        z = torch.empty((B, model.d), dtype=torch.int32, device=x_u8.device)
    if prior is None and want_prior and model.d_fact:
        prior = torch.empty((B, 2, model.d_fact), dtype=torch.int32, device=x_u8.device)
    rc = load_library().iodf_forward(model.handle, _ptr(x_u8), B, _ptr(z), _ptr(prior), _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_forward")
    return z, prior


def iodf_inverse(model, z, x_u8=None, prior=None, out_of_range=None, stream=None):
    """z: cuda int32 [B,d]. Returns x_u8 uint8 [B,C,H,W]."""
    import torch
    B = z.shape[0]
    assert z.is_cuda and z.dtype == torch.int32 and z.is_contiguous()
    if x_u8 is None:
        x_u8 = torch.empty((B,) + tuple(model.in_shape), dtype=torch.uint8, device=z.device)
    rc = load_library().iodf_inverse(model.handle, _ptr(z), B, _ptr(x_u8), _ptr(prior), _ptr(out_of_range),
                                     _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_inverse")
    return x_u8


IODF_LEVEL_PRIOR = 1
IODF_LEVEL_COUPLINGS = 2


def iodf_inverse_level(model, level, phase, z, x_u8=None, prior=None, out_of_range=None, stream=None):
    """One step of the level-stepped decode (see include/iodf.h). z: cuda int32 [B,d] (full size)."""
    rc = load_library().iodf_inverse_level(model.handle, level, phase, _ptr(z), z.shape[0], _ptr(x_u8), _ptr(prior),
                                           _ptr(out_of_range), _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_inverse_level")


def iodf_forward_patches(model, image_u8, z=None, prior=None, stream=None):
    """image_u8: cuda uint8 [C,H,W], H and W multiples of the model's input size. Returns (z, prior)
    of the batch of patches in row-major patch order."""
    import torch
    _, H, W = image_u8.shape
    B = (H // model.in_shape[1]) * (W // model.in_shape[2])
    if z is None:
        z = torch.empty((B, model.d), dtype=torch.int32, device=image_u8.device)
    if prior is None and model.d_fact:
        prior = torch.empty((B, 2, model.d_fact), dtype=torch.int32, device=image_u8.device)
    rc = load_library().iodf_forward_patches(model.handle, _ptr(image_u8), H, W, _ptr(z), _ptr(prior), _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_forward_patches")
    return z, prior


def iodf_inverse_patches(model, z, H, W, image_u8=None, prior=None, out_of_range=None, stream=None):
    """z: cuda int32 [B,d] of the patch batch. Returns the image uint8 [C,H,W]."""
    import torch
    if image_u8 is None:
        image_u8 = torch.empty((model.in_shape[0], H, W), dtype=torch.uint8, device=z.device)
    rc = load_library().iodf_inverse_patches(model.handle, _ptr(z), H, W, _ptr(image_u8), _ptr(prior),
                                             _ptr(out_of_range), _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_inverse_patches")
    return image_u8


class Codec:
    """Handle of an iodf_codec; destroyed when garbage collected."""

    def __init__(self, handle, layout, model):
        self.handle, self.layout, self.model = handle, layout, model
        self.n_blocks, self.n_streams = int(layout.n_blocks), int(layout.n_streams)
        self.words_per_stream = int(layout.words_per_stream)

    def __del__(self):
        h, self.handle = getattr(self, "handle", None), None
        if h and _lib is not None:
            _lib.iodf_codec_destroy(h)


def iodf_codec_create(model, codec):
    """codec: dict with the tables G (uint16), R (uint32), umax, final_ls, elems_per_stream."""
    L = load_library()
    G = np.ascontiguousarray(codec["G"], dtype=np.uint16)
    R = np.ascontiguousarray(codec["R"], dtype=np.uint32)
    desc = CodecDesc(IODF_ABI_VERSION, G.ctypes.data, int(codec["umax"]), R.ctypes.data, len(R),
                     int(codec["final_ls"]), int(codec["elems_per_stream"]))
    out = C.c_void_p()
    rc = L.iodf_codec_create(model.handle, C.byref(desc), C.byref(out))
    if rc != 0:
        raise IodfError(rc, "iodf_codec_create")
    lay = CodecLayout()
    L.iodf_codec_get_layout(out, C.byref(lay))
    return Codec(out, lay, model)


def iodf_rans_encode(codec, z, prior, words=None, counts=None, stream=None):
    """z cuda int32 [B,d], prior cuda int32 [B,2,d_fact] -> (words uint16 [B,S,cap], counts uint32-as-int32 [B,S])."""
    import torch
    B = z.shape[0]
    if words is None:
        words = torch.empty((B, codec.n_streams, codec.words_per_stream), dtype=torch.int16, device=z.device)
    if counts is None:
        counts = torch.empty((B, codec.n_streams), dtype=torch.int32, device=z.device)
    rc = load_library().iodf_rans_encode(codec.handle, _ptr(z), _ptr(prior), B, _ptr(words), _ptr(counts), _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_rans_encode")
    return words, counts


def iodf_rans_decode_block(codec, block, words, counts, prior, z, stream=None):
    rc = load_library().iodf_rans_decode_block(codec.handle, int(block), _ptr(words), _ptr(counts), _ptr(prior),
                                               z.shape[0], _ptr(z), _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_rans_decode_block")


def iodf_rans_packed_capacity(codec, B):
    return int(load_library().iodf_rans_packed_capacity(codec.handle, int(B)))


def iodf_rans_pack(codec, words, counts, packed=None, stream=None):
    """Container -> compact byte stream. Returns (packed cuda uint8 tensor of full capacity, total bytes);
    reading the total synchronises."""
    import torch
    B = counts.shape[0]
    if packed is None:
        packed = torch.empty(iodf_rans_packed_capacity(codec, B), dtype=torch.uint8, device=counts.device)
    rc = load_library().iodf_rans_pack(codec.handle, _ptr(words), _ptr(counts), B, _ptr(packed), _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_rans_pack")
    payload = int(packed[4 * B:4 * B + 4].cpu().numpy().view(np.uint32)[0])
    return packed, 4 * (B + 1) + payload


def iodf_rans_unpack(codec, packed, nbytes, B, words=None, counts=None, stream=None):
    import torch
    if words is None:
        words = torch.zeros((B, codec.n_streams, codec.words_per_stream), dtype=torch.int16, device=packed.device)
    if counts is None:
        counts = torch.zeros((B, codec.n_streams), dtype=torch.int32, device=packed.device)
    rc = load_library().iodf_rans_unpack(codec.handle, _ptr(packed), int(nbytes), int(B), _ptr(words), _ptr(counts),
                                         _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_rans_unpack")
    return words, counts


def iodf_compress_host(model, codec, x_u8_host, out_host=None, stream=None):
    """Host uint8 images [B,C,H,W] -> (host uint8 buffer, number of valid bytes). Synchronises."""
    import torch
    B = x_u8_host.shape[0]
    if out_host is None:
        out_host = torch.empty(iodf_rans_packed_capacity(codec, B), dtype=torch.uint8).pin_memory()
    n = C.c_size_t(0)
    rc = load_library().iodf_compress_host(model.handle, codec.handle, _ptr(x_u8_host), B, _ptr(out_host),
                                           out_host.numel(), C.byref(n), _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_compress_host")
    return out_host, int(n.value)


def iodf_decompress_host(model, codec, in_host, nbytes, B, x_u8_host=None, stream=None):
    """Compact byte stream (host) -> host uint8 images; valid after the stream is synchronised."""
    import torch
    if x_u8_host is None:
        x_u8_host = torch.empty((B,) + tuple(model.in_shape), dtype=torch.uint8).pin_memory()
    rc = load_library().iodf_decompress_host(model.handle, codec.handle, _ptr(in_host), int(nbytes), int(B),
                                             _ptr(x_u8_host), _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_decompress_host")
    return x_u8_host


def iodf_codec_check(codec, stream=None):
    n = C.c_uint32(0)
    rc = load_library().iodf_codec_check(codec.handle, _stream(stream), C.byref(n))
    if rc != 0:
        raise IodfError(rc, "iodf_codec_check (%d streams)" % n.value)


def iodf_forward_host(model, x_u8, z, prior=None, stream=None):
    """Host (ideally pinned) torch tensors in and out; results valid after the stream is synchronised."""
    rc = load_library().iodf_forward_host(model.handle, _ptr(x_u8), x_u8.shape[0], _ptr(z), _ptr(prior),
                                          _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_forward_host")


def iodf_inverse_host(model, z, x_u8, stream=None):
    rc = load_library().iodf_inverse_host(model.handle, _ptr(z), z.shape[0], _ptr(x_u8), _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_inverse_host")


def iodf_forward_timed(model, x_u8, z, prior=None, stream=None):
    """Encode with per-level event timing; returns the list of per-level kernel times in ms."""
    n = int(model.layout.n_levels)
    ms = (C.c_float * n)()
    rc = load_library().iodf_forward_timed(model.handle, _ptr(x_u8), x_u8.shape[0], _ptr(z), _ptr(prior),
                                           _stream(stream), ms)
    if rc != 0:
        raise IodfError(rc, "iodf_forward_timed")
    return list(ms)


def iodf_inverse_timed(model, z, x_u8, prior=None, out_of_range=None, stream=None):
    n = int(model.layout.n_levels)
    ms = (C.c_float * n)()
    rc = load_library().iodf_inverse_timed(model.handle, _ptr(z), z.shape[0], _ptr(x_u8), _ptr(prior),
                                           _ptr(out_of_range), _stream(stream), ms)
    if rc != 0:
        raise IodfError(rc, "iodf_inverse_timed")
    return list(ms)


IODF_STATIC_SCRATCH_BYTES = 8 * 1024 * 1024


def iodf_static_scratch_bytes_per_image(model):
    return int(load_library().iodf_static_scratch_bytes_per_image(model.handle))


def iodf_forward_static(model, x_u8, z, prior=None, stream=None):
    """Encode using the library's fixed scratch array instead of the model's allocated workspace.
    The caller passes every buffer (this wrapper allocates nothing either)."""
    rc = load_library().iodf_forward_static(model.handle, _ptr(x_u8), x_u8.shape[0], _ptr(z), _ptr(prior),
                                            _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_forward_static")


def iodf_check(model, stream=None):
    rc = load_library().iodf_check(model.handle, _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_check")


def iodf_selftest_timeout(model, tries=3, stream=None):
    rc = load_library().iodf_selftest_timeout(model.handle, int(tries), _stream(stream))
    if rc != 0:
        raise IodfError(rc, "iodf_selftest_timeout")


def iodf_int8_mma_peak(model, mma_groups, stream=None):
    """Enqueue the MMA-only kernel; returns the int8 OPs of the launch."""
    ops = C.c_ulonglong(0)
    rc = load_library().iodf_int8_mma_peak(model.handle, int(mma_groups), _stream(stream), C.byref(ops))
    if rc != 0:
        raise IodfError(rc, "iodf_int8_mma_peak")
    return int(ops.value)


def iodf_level_kernel_name(model, level):
    return load_library().iodf_level_kernel_name(model.handle, int(level)).decode()


def iodf_launches_per_call(model, inverse=False):
    return load_library().iodf_launches_per_call(model.handle, int(inverse))


def iodf_level_images_per_cta(model, level):
    n = load_library().iodf_level_images_per_cta(model.handle, int(level))
    if n < 0:
        raise IodfError(n, "iodf_level_images_per_cta")
    return n
