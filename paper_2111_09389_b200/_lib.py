"""ctypes loader of liblpdt.so.  There is no fallback: a missing or unloadable
library raises."""
import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
SO_PATH = os.path.join(HERE, "liblpdt.so")

_lib = None

_vp, _i32, _i64, _u32, _u64, _f32, _sz = (C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_uint64,
                                          C.c_float, C.c_size_t)


class ConvDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("nodes", "B", "H", "W", "Cin", "Cout", "R", "S", "stride", "pad")]


# name -> (restype, argtypes); mirrors include/lpdt.h
SIGNATURES = {
    "lpdt_version": (C.c_char_p, []),
    "lpdt_status_string": (C.c_char_p, [_i32]),
    "lpdt_last_kernel": (C.c_char_p, []),
    "lpdt_launch_count": (_u64, []),
    "lpdt_fill_zero": (_i32, [_vp, _sz, _vp]),
    "lpdt_check_status": (_i32, [_vp, _vp]),
    "lpdt_selftest_bounded_wait": (_i32, [_u64, _vp, _vp, _vp]),
    "lpdt_message_bytes": (_i64, [_i64, _i32, _vp, _vp, _i32, _i32]),
    "lpdt_quantize_workspace_size": (_sz, [_i32]),
    "lpdt_quantize": (_i32, [_vp, _i32, _i64, _i64, _i32, _i32, _u64, _u32, _vp, _vp, _vp, _vp, _sz, _vp]),
    "lpdt_quantize_static": (_i32, [_vp, _i32, _i64, _i64, _i32, _i32, _u64, _u32, _vp, _vp, _vp, _vp]),
    "lpdt_quantize_with_range": (_i32, [_vp, _i32, _i64, _i64, _vp, _i32, _u64, _u32, _vp, _vp, _vp]),
    "lpdt_quantize_batch_workspace_size": (_sz, [_i32, _i32]),
    "lpdt_quantize_batch": (_i32, [_vp, _i32, _i64, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "lpdt_dequantize": (_i32, [_vp, _i32, _i64, _vp, _vp, _vp, _i64, _vp]),
    "lpdt_qconv_workspace_size": (_sz, [C.POINTER(ConvDesc), _i32]),
    "lpdt_qconv_fwd": (_i32, [C.POINTER(ConvDesc), _vp, _vp, _vp, _vp, _vp, _i64, _vp, _vp, _vp, _sz, _vp, _vp]),
    "lpdt_qconv_fwd_affine_workspace_size": (_sz, [C.POINTER(ConvDesc)]),
    "lpdt_qconv_fwd_affine": (_i32, [C.POINTER(ConvDesc), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _vp, _vp, _vp, _sz,
                                     _vp, _vp]),
    "lpdt_qconv_bwd_data_affine_workspace_size": (_sz, [C.POINTER(ConvDesc)]),
    "lpdt_qconv_bwd_data_affine": (_i32, [C.POINTER(ConvDesc), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _vp]),
    "lpdt_qconv_bwd_weight_affine_workspace_size": (_sz, [C.POINTER(ConvDesc)]),
    "lpdt_qconv_bwd_weight_affine": (_i32, [C.POINTER(ConvDesc), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _vp, _vp, _sz,
                                            _vp, _vp]),
    "lpdt_qconv_bwd_data": (_i32, [C.POINTER(ConvDesc), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _vp]),
    "lpdt_qconv_bwd_weight": (_i32, [C.POINTER(ConvDesc), _vp, _vp, _vp, _vp, _vp, _i64, _vp, _vp, _sz, _vp, _vp]),
    "lpdt_range_evonorm_fwd": (_i32, [_i32] * 6 + [_f32] + [_vp] * 4 + [_i64] + [_vp] * 7 + [_vp]),
    "lpdt_range_evonorm_q8_ctl_size": (_sz, [_i32]),
    "lpdt_range_evonorm_fwd_q8_fits": (_i32, [_i32] * 5),
    "lpdt_range_evonorm_fwd_q8": (_i32, [_i32] * 6 + [_f32] + [_vp] * 4 + [_i64] + [_vp] * 9 + [_vp, _sz, _vp, _vp]),
    "lpdt_range_evonorm_bwd_q8_fits": (_i32, [_i32] * 5),
    "lpdt_range_evonorm_bwd_q8": (_i32, [_i32] * 6 + [_f32] + [_vp] * 4 + [_i64] + [_vp] * 9 +
                                  [_i64, _vp, _vp, _sz, _vp, _sz, _vp, _vp]),
    "lpdt_range_evonorm_bwd_workspace_size": (_sz, [_i32, _i32, _i32]),
    "lpdt_range_evonorm_bwd": (_i32, [_i32] * 6 + [_f32] + [_vp] * 4 + [_i64] + [_vp] * 8 + [_i64, _vp, _vp, _sz, _vp]),
    "lpdt_evonorm_s0_fwd": (_i32, [_i32] * 6 + [_f32] + [_vp] * 4 + [_i64] + [_vp] * 4),
    "lpdt_evonorm_s0_bwd_workspace_size": (_sz, [_i32, _i32, _i32]),
    "lpdt_evonorm_s0_bwd": (_i32, [_i32] * 6 + [_f32] + [_vp] * 4 + [_i64] + [_vp] * 6 + [_i64, _vp, _sz, _vp]),
    "lpdt_range_bn_workspace_size": (_sz, [_i32, _i32]),
    "lpdt_range_bn_fwd": (_i32, [_i32] * 5 + [_f32] + [_vp] * 3 + [_i64] + [_vp] * 6 + [_vp, _sz, _vp]),
    "lpdt_range_bn_bwd": (_i32, [_i32] * 5 + [_f32] + [_vp] * 3 + [_i64] + [_vp] * 8 + [_i64, _vp, _sz, _vp]),
    "lpdt_range_evonorm_bwd_params_batch": (_i32, [_i32, _i32, _i32, _vp, _vp, _vp, _vp, _i64, _vp]),
    "lpdt_dequantize_acc_batch": (_i32, [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _vp]),
    "lpdt_range_evonorm_bwd_params": (_i32, [_i32, _i32, _i32, _vp, _sz, _vp, _vp, _vp, _i64, _vp]),
    "lpdt_gossip_mix_workspace_size": (_sz, [_i32, _i64, _i32]),
    "lpdt_gossip_mix": (_i32, [_i32, _i64, _vp, _vp, _vp, _vp, _f32, _i32, _vp, _vp, _vp, _sz, _vp, _vp]),
    "lpdt_gossip_mix_q8": (_i32, [_i32, _i64, _vp, _vp, _vp, _vp, _f32, _i32, _vp, _vp, _vp, _vp, _sz, _vp, _vp]),
    "lpdt_deepsqueeze_mix": (_i32, [_i32, _i64, _vp, _vp, _vp, _vp, _f32, _i32, _vp, _vp, _i32, _vp, _vp, _sz, _vp,
                                    _vp]),
    "lpdt_sgd_gossip_mix": (_i32, [_i32, _i64, _vp, _vp, _f32, _vp, _vp, _vp, _vp, _f32, _vp]),
    "lpdt_pushsum_debias": (_i32, [_i32, _i64, _vp, _vp, _vp, _f32, _vp, _vp, _vp]),
    "lpdt_sgd_update": (_i32, [_i64, _vp, _vp, _f32, _vp, _vp]),
    "lpdt_residual_add": (_i32, [_i32] * 8 + [_vp] * 5),
    "lpdt_residual_add_bwd": (_i32, [_i32] * 8 + [_vp] * 4),
    "lpdt_avgpool": (_i32, [_i32] * 4 + [_vp] * 3),
    "lpdt_avgpool_bwd": (_i32, [_i32] * 4 + [_vp] * 3),
    "lpdt_maxpool2x2": (_i32, [_i32] * 5 + [_vp] * 4),
    "lpdt_maxpool2x2_bwd": (_i32, [_i32] * 5 + [_vp] * 4),
    "lpdt_softmax_ce": (_i32, [_i32] * 3 + [_vp] * 6),
    "lpdt_colsum": (_i32, [_i32] * 3 + [_vp, _vp, _i64, _vp]),
}


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(SO_PATH):
            raise RuntimeError(
                f"{SO_PATH} is missing: build it with `python -m paper_2111_09389_b200.build`; "
                "there is no CPU or library fallback")
        _lib = C.CDLL(SO_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(_lib, name)
            fn.restype = res
            fn.argtypes = args
    return _lib
