#pragma once
#include "mask.cuh"
#include "ptx.cuh"
