"""HAC / sHAC compressed-domain products on NVIDIA B200: Python binding of libhac_b200.so.

The functions carry the names of the C ABI (include/hac.h) and only marshal arguments."""
from .binding import (Format, HacError, chain as hac_chain, build_unified as hac_build_unified, QUANT_GRID, QUANT_KMEANS, QUANT_NONE, QUANT_PWS, QUANT_UNIFORM, EXPORTS, load,
                      library_path)


def hac_build(W, **params) -> Format:
    """hac_build of the C ABI: prune, share weights, Huffman-code every entry of W (HAC)."""
    return Format("hac", W, **params)


def shac_build(W, **params) -> Format:
    """shac_build of the C ABI: prune, share weights, CSC with Huffman-coded nz (sHAC)."""
    return Format("shac", W, **params)


def hac_dot(fmt: Format, x, y=None, workspace=None, layout="nb"):
    """hac_dot of the C ABI: y = W^T x on the device from the HAC stream."""
    assert fmt.kind == "hac"
    return fmt.dot(x, y, workspace, layout)


def shac_dot(fmt: Format, x, y=None, workspace=None, layout="nb"):
    """shac_dot of the C ABI: y = W^T x on the device from the sHAC arrays."""
    assert fmt.kind == "shac"
    return fmt.dot(x, y, workspace, layout)


__all__ = ["Format", "HacError", "QUANT_NONE", "QUANT_KMEANS", "QUANT_UNIFORM", "QUANT_GRID", "QUANT_PWS", "EXPORTS", "load",
           "library_path", "hac_build", "shac_build", "hac_dot", "shac_dot", "hac_chain", "hac_build_unified"]
