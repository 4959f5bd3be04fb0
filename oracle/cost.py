"""Cost identity of Sec. 4.1: BOPs = FLOPs * b_w * b_a.  Test infrastructure only."""


def bops(flops, b_w, b_a):
    """Bit operations of a layer (or model) with `flops` operations at b_w-bit weights, b_a-bit activations."""
    return flops * b_w * b_a


def table_bytes(T, groups, scalars_per_group, bytes_per_scalar=1):
    """Size of the per-timestep parameter sets S, Z of Eq. 7."""
    return T * groups * scalars_per_group * bytes_per_scalar
